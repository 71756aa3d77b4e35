"""Small-footprint driver of the decode step for profiling one kernel at a time.

    python -m paper_2401_10774_b200.microbench [--model 7b] [--layers 2] [--prompt 512] [--steps 3] [--L-max 4096]
    python -m paper_2401_10774_b200.microbench --attention 4096 [--model 7b] [--caches 32] [--steps 5]

Builds a model of the named width with only a few decoder layers (a couple of GB on the device, more than
the L2), prefills a seeded prompt and runs a few tree-verification steps through the C ABI.  Meant to be run
under a profiler restricted to one kernel; prints per-category device times from the library's own events.
`--attention L` times the stand-alone `tree_attention` entry instead: `--caches` launches over that many distinct
K/V caches of length L (together larger than the L2) per repetition, replayed from a CUDA graph.
`--heads-train N` times the forward/backward pass of the heads' training objective over N positions (one head unless
`--heads K`), and reports it against the measured dense bf16 throughput.

    python -m paper_2401_10774_b200.microbench --heads-train 4096 [--model 7b] [--heads 1] [--steps 3]
"""
from __future__ import annotations

import argparse
import json

import numpy as np


def main():
    import torch

    from . import binding as B
    from . import inputs as I

    ap = argparse.ArgumentParser()
    ap.add_argument("--model", default="7b")
    ap.add_argument("--layers", type=int, default=2)
    ap.add_argument("--prompt", type=int, default=512)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3, help="untimed steps first (the library captures its step graph on the second)")
    ap.add_argument("--L-max", type=int, default=4096)
    ap.add_argument("--tree", default=None)
    ap.add_argument("--profile-events", action="store_true", help="time every launch with CUDA events")
    ap.add_argument("--typical", action="store_true", help="typical acceptance (0.7 / 0.09 / 0.3) instead of greedy")
    ap.add_argument("--attention", type=int, default=0, metavar="L", help="time tree_attention alone at cache length L")
    ap.add_argument("--caches", type=int, default=32)
    ap.add_argument("--planes", type=int, default=2, choices=(1, 2))
    ap.add_argument("--attention-kernel", type=int, default=0, choices=(0, 1, 2), help="0 automatic, 1 mma.sync, 2 tcgen05")
    ap.add_argument("--no-graphs", action="store_true", help="launch every step kernel by kernel")
    ap.add_argument("--pack-weights", type=int, default=-1, choices=(-1, 0, 1), help="weights re-laid tile by tile (1) or streamed as given (0); -1: the library's default")
    ap.add_argument("--device-weights", action="store_true",
                    help="draw the weights on the device (N(0, 0.02^2), not the seeded host recipe): seconds instead of a "
                         "minute of set-up, for timing runs whose numbers do not depend on the values")
    ap.add_argument("--heads-train", type=int, default=0, metavar="N", help="time the heads' training pass over N positions")
    ap.add_argument("--heads", type=int, default=1, help="heads in the training pass")
    args = ap.parse_args()
    if args.attention:
        return attention_only(args)
    if args.heads_train:
        return heads_train_only(args)

    cfg = I.model_shape(args.model, n_layers=args.layers)
    tree_name = args.tree or ("sparse64_d5" if cfg["n_medusa"] >= 5 else "sparse64_d4")
    spec = I.LARGE_TREE_SPECS[tree_name] if tree_name in I.LARGE_TREE_SPECS else I.TREE_SPECS[tree_name]
    cfg["max_tree_nodes"] = spec["n_nodes"]
    if args.device_weights:
        gen = torch.Generator(device="cuda").manual_seed(40)

        def rnd(*shape, std=0.02, mean=0.0):
            return (torch.randn(*shape, device="cuda", generator=gen) * std + mean).bfloat16()

        d, F, V, K = cfg["d"], cfg["ffn"], cfg["vocab"], cfg["n_medusa"]
        hd, hkd = cfg["n_heads"] * cfg["head_dim"], I.kv_heads(cfg) * cfg["head_dim"]
        dw = dict(embed=rnd(V, d), lm_head=rnd(V, d), final_norm=rnd(d, std=0.0, mean=1.0), medusa_w1=rnd(K, d, d),
                  medusa_w2=rnd(K, V, d), layers=[])
        for _ in range(cfg["n_layers"]):
            dw["layers"].append(dict(attn_norm=rnd(d, std=0.0, mean=1.0), wq=rnd(hd, d), wk=rnd(hkd, d), wv=rnd(hkd, d),
                                     wo=rnd(d, hd), ffn_norm=rnd(d, std=0.0, mean=1.0), w_gate=rnd(F, d), w_up=rnd(F, d),
                                     w_down=rnd(d, F)))
    else:
        w = I.make_weights(cfg, seed=40, dtype="bf16")

        def dev(a):
            return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda().view(torch.bfloat16)

        dw = {k: dev(v) for k, v in w.items() if k != "layers"}
        dw["layers"] = [{k: dev(v) for k, v in lw.items()} for lw in w["layers"]]
    ctx = B.Context(cfg, B.BF16, args.L_max)
    ctx.build_tree_buffers(B.default_tree_paths(spec["per_depth_topk"], spec["n_nodes"]))
    if args.planes != 2:
        ctx.set_option(B.OPT_ACTIVATION_PLANES, args.planes)
    if args.attention_kernel:
        ctx.set_option(B.OPT_ATTENTION_KERNEL, args.attention_kernel)
    if args.no_graphs:
        ctx.set_option(B.OPT_STEP_GRAPHS, 0)
    if args.pack_weights >= 0:
        ctx.set_option(B.OPT_PACK_WEIGHTS, args.pack_weights)
    ctx.load_weights(dw)
    # a cache of the requested length without paying for a long prefill: prefill 64 tokens, then tell the
    # library the rest is there (the K/V values beyond are zeros, which is fine for timing)
    prompt = I.make_prompt(args.prompt, cfg["vocab"], 41)
    ctx.prefill(torch.from_numpy(prompt).cuda())
    torch.cuda.synchronize()
    params = (B.AcceptParams(mode=B.TYPICAL, temperature=0.7, eps=0.09, delta=0.3) if args.typical
              else B.AcceptParams(mode=B.GREEDY))
    if args.profile_events:
        ctx.get_profile(reset=True)
        ctx.set_profiling(True)
    for _ in range(args.warmup):
        ctx.decode_step(params)
    if args.profile_events:
        ctx.get_profile(reset=True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        ctx.decode_step(params)
    e1.record()
    torch.cuda.synchronize()
    out = dict(model=args.model, layers=args.layers, steps=args.steps, cache_len=ctx.state()["cache_len"],
               ms_per_step=e0.elapsed_time(e1) / args.steps, status=ctx.device_status(), step_graphs=ctx.step_graph_info())
    if args.profile_events:
        out["kernels"] = {k: dict(ms_per_step=v["ms"] / args.steps, launches_per_step=v["launches"] / args.steps)
                          for k, v in ctx.get_profile().items() if v["launches"]}
    print(json.dumps(out))
    ctx.close()


def attention_only(args):
    import torch

    from . import binding as B
    from . import inputs as I
    from . import roofline as R

    shape = I.model_shape(args.model, n_layers=0)
    H, D, L, T = shape["n_heads"], shape["head_dim"], args.attention, 64
    st = torch.cuda.Stream()
    cfg = dict(n_layers=0, d=H * D, n_heads=H, head_dim=D, ffn=8, vocab=8, n_medusa=4)
    ctx = B.Context(cfg, B.BF16, max(L, 64), stream=st.cuda_stream)
    spec = I.TREE_SPECS["sparse64_d4"]
    ctx.build_tree_buffers(B.default_tree_paths(spec["per_depth_topk"], spec["n_nodes"]))
    g = torch.Generator(device="cuda").manual_seed(7)
    rnd = lambda *sh: torch.randn(*sh, device="cuda", generator=g).bfloat16()
    q, kn, vn = rnd(T, H, D), rnd(T, H, D), rnd(T, H, D)
    kcs = [rnd(H, max(L, 64), D) for _ in range(args.caches)]
    vcs = [rnd(H, max(L, 64), D) for _ in range(args.caches)]
    out = torch.zeros_like(q)
    cl = torch.tensor([L], dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()

    def sweep():
        for kc, vc in zip(kcs, vcs):
            ctx.tree_attention(q, kn, vn, kc, vc, cl, False, out)

    with torch.cuda.stream(st):
        sweep()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=st):
        sweep()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(st):
        graph.replay()
        e0.record(st)
        for _ in range(args.steps):
            graph.replay()
        e1.record(st)
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / (args.steps * args.caches)
    nbytes = R.attention_bytes(T, H, D, L)  # K and V of the cache; q, tree k, tree v, output
    peak, src = R.hbm_peak_gbs()
    print(json.dumps(dict(op="tree_attention", model=args.model, L=L, T=T, H=H, us_per_launch=round(us, 2),
                          achieved_gbs=round(nbytes / us / 1e3, 1), frac=round(nbytes / us / 1e3 / peak, 3), peak_gbs=peak,
                          peak_source=src, status=ctx.device_status())))
    ctx.close()


def heads_train_only(args):
    import torch

    from . import binding as B
    from . import inputs as I
    from . import roofline as R

    shape = I.model_shape(args.model, n_layers=0)
    d, V, K, N = shape["d"], shape["vocab"], args.heads, args.heads_train
    cfg = dict(n_layers=0, d=d, n_heads=shape["n_heads"], head_dim=shape["head_dim"], ffn=8, vocab=V, n_medusa=K)
    gen = torch.Generator(device="cuda").manual_seed(1)
    rnd = lambda *sh: (torch.randn(*sh, device="cuda", generator=gen) * 0.02).bfloat16()
    w = dict(embed=rnd(V, d), lm_head=rnd(V, d), final_norm=torch.ones(d, device="cuda").bfloat16(), layers=[],
             medusa_w1=rnd(K, d, d), medusa_w2=rnd(K, V, d))
    ctx = B.Context(cfg, B.BF16, 64)
    ctx.load_weights(w)
    h = torch.randn(N, d, device="cuda", generator=gen).bfloat16()
    y = torch.randint(0, V, (K, N), device="cuda", dtype=torch.int32)
    loss = torch.zeros(K + 1, device="cuda")
    g1, g2 = torch.zeros(K, d, d, device="cuda"), torch.zeros(K, V, d, device="cuda")
    for _ in range(max(args.warmup, 1)):
        ctx.heads_loss_and_grads(h, y, loss, g1, g2)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        ctx.heads_loss_and_grads(h, y, loss, g1, g2)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    flop = K * N * (4.0 * d * d + 6.0 * V * d)  # five projections per head and position
    peak, src = R.tensor_peak_tflops()
    print(json.dumps(dict(op="heads_loss_and_grads", model=args.model, heads=K, positions=N, ms_per_pass=round(ms, 3),
                          positions_per_s=round(N / ms * 1e3), tflops=round(flop / ms / 1e9, 1), frac=round(flop / ms / 1e9 / peak, 3),
                          peak_tflops=peak, peak_source=src, loss=[round(float(v), 4) for v in loss.cpu()], status=ctx.device_status())))
    ctx.close()


if __name__ == "__main__":
    main()
