#!/usr/bin/env python
"""Benchmark of the Medusa tree-verification decode step (7B shape, bf16, batch 1) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

A step is one full pass of the hot path: Medusa heads + top-k + candidate expansion, the backbone over the
64-node tree with tree attention against the KV cache, acceptance, KV commit.  Prints ONE JSON line.
The step replicates without communication, so --gpus N runs N independent replicas (one process per GPU).
`--impl reference` times the CPU oracle (a deliberately plain program) on the same workload description.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2401_10774_b200 import inputs as I  # noqa: E402
from paper_2401_10774_b200 import roofline as R  # noqa: E402

# The default (and the headline) is the 7B greedy step; `--workload 13b` measures the 13B-shape step with five
# heads, the depth-5 tree, typical acceptance with a Gumbel-sampled root and a 3584-token prompt; `--workload 7b_long`
# is the 7B step against a nearly full cache (3840-token prompt, capacity 4096); `--workload mistral7b` is the shape of
# the paper's Zephyr-7B backbone (grouped-query attention, 8 key/value heads) with five heads and typical acceptance;
# `--workload 7b_tree128 / 7b_tree256` are the 7B step with larger trees.
WORKLOADS = {
    "7b": dict(name="7b_medusa1_greedy_step", model="7b", tree="sparse64_d4", prompt=512, L_max=4096, weights_seed=40,
               prompt_seed=41, mode="greedy", oracle_layers=8,
               metric="decode tokens/s (7B-shape bf16 Medusa tree-verification step, 64-node tree, batch 1)"),
    "7b_long": dict(name="7b_medusa1_greedy_step_long_cache", model="7b", tree="sparse64_d4", prompt=3840, L_max=4096,
                    weights_seed=40, prompt_seed=41, mode="greedy", oracle_layers=4,
                    metric="decode tokens/s (7B-shape bf16 Medusa tree-verification step, 64-node tree, batch 1, "
                           "cache of 3.8-4.1 K tokens)"),
    "mistral7b": dict(name="mistral7b_gqa_medusa_typical_step", model="mistral7b", tree="sparse64_d5", prompt=1024, L_max=4096,
                      weights_seed=60, prompt_seed=61, noise_seed=62, mode="typical", temperature=0.7, eps=0.09, delta=0.3,
                      oracle_layers=4,
                      metric="decode tokens/s (Mistral-7B-shape bf16 Medusa tree-verification step, grouped-query attention "
                             "with 8 key/value heads, 5 heads, 64-node depth-5 tree, typical acceptance, batch 1)"),
    # trees of more than 64 nodes (the paper's Fig. 4 studies up to 256): the same 7B step with the 128- / 256-node
    # surrogate trees; the token rows are processed in tiles of 64, the weights streamed once per tile
    "7b_tree128": dict(name="7b_medusa1_greedy_step_tree128", model="7b", tree="sparse128_d4", prompt=512, L_max=4096,
                       weights_seed=40, prompt_seed=41, mode="greedy", oracle_layers=2,
                       metric="decode tokens/s (7B-shape bf16 Medusa tree-verification step, 128-node tree, batch 1)"),
    "7b_tree256": dict(name="7b_medusa1_greedy_step_tree256", model="7b", tree="sparse256_d4", prompt=512, L_max=4096,
                       weights_seed=40, prompt_seed=41, mode="greedy", oracle_layers=1,
                       metric="decode tokens/s (7B-shape bf16 Medusa tree-verification step, 256-node tree, batch 1)"),
    # batch > 1: four sequences (own caches, prompts of 512 tokens from four seeds) stepped in one backbone pass
    "7b_batch4": dict(name="7b_medusa1_greedy_step_batch4", model="7b", tree="sparse64_d4", prompt=512, L_max=4096,
                      weights_seed=40, prompt_seed=41, mode="greedy", oracle_layers=2, batch=4,
                      metric="decode tokens/s, all sequences (7B-shape bf16 Medusa tree-verification step, 64-node tree, batch 4)"),
    "13b": dict(name="13b_medusa_typical_step", model="13b", tree="sparse64_d5", prompt=3584, L_max=4096, weights_seed=50,
                prompt_seed=51, noise_seed=52, mode="typical", temperature=0.7, eps=0.09, delta=0.3, oracle_layers=4,
                metric="decode tokens/s (13B-shape bf16 Medusa tree-verification step, 64-node depth-5 tree, typical "
                       "acceptance, batch 1)"),
}
WORKLOAD = WORKLOADS["7b"]


def tree_spec(name: str) -> dict:
    return I.LARGE_TREE_SPECS[name] if name in I.LARGE_TREE_SPECS else I.TREE_SPECS[name]


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap,timestamp")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            f = tempfile.NamedTemporaryFile("w", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "25"], stdout=f,
                                         stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self, t_load0=None, t_load1=None) -> dict:
        """Summary of the samples stamped inside the host-clock window [t_load0, t_load1] (the GPU under load)."""
        import datetime

        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.05)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in open(self.path):
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                if t_load0 is not None and len(parts) >= 9:
                    ts = datetime.datetime.strptime(parts[8], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    if ts < t_load0 + 0.03 or ts > t_load1:
                        continue  # the GPU was idle (or just ramping) when this sample was taken
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        os.unlink(self.path)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no samples"])
        return dict(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))


# ----------------------------------------------------------------------------------------------- CPU oracle legs

class OracleSample:
    """The oracle, as it stands, on a bounded sample of one tree-verification step: Medusa heads + top-k and
    LM head + acceptance run in full; `n_sample_layers` of the identical decoder layers are run at T=64 against
    a cache of length L and the layer time is multiplied up to the full depth."""

    def __init__(self, n_sample_layers: int, cfg_full: dict, L: int):
        from oracle import medusa_oracle as O

        self.O = O
        self.n = n_sample_layers
        self.cfg_full = cfg_full
        self.L = L
        spec = tree_spec(WORKLOAD["tree"])
        self.tree = O.build_tree_buffers(O.default_tree_paths(spec["per_depth_topk"], spec["n_nodes"]))
        cfg = dict(cfg_full, n_layers=n_sample_layers)
        self.w = I.make_weights(cfg, seed=WORKLOAD["weights_seed"], dtype="bf16")
        self.model = O.Model(cfg, self.w)
        self.model0 = O.Model(dict(cfg_full, n_layers=0), dict(self.w, layers=[]))
        g = I.rng(WORKLOAD["prompt_seed"], "oracle-sample")
        self.kc = g.standard_normal(self.model.cache_shape(L + 64))
        self.vc = g.standard_normal(self.model.cache_shape(L + 64))
        self.kc0 = np.zeros(self.model0.cache_shape(8))
        self.tok = g.integers(0, cfg["vocab"], size=self.tree["T"]).astype(np.int32)
        self.h = g.standard_normal(cfg["d"])
        self.cores = int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))

    def run(self):
        """-> (seconds for a full-depth step, description)"""
        O, tree = self.O, self.tree
        t0 = time.perf_counter()
        x, z = O.medusa_heads(self.h, self.w["medusa_w1"], self.w["medusa_w2"])
        for k in range(self.cfg_full["n_medusa"]):
            O.topk(z[k].astype(np.float32), tree["topk"])
        t_heads = time.perf_counter() - t0
        t0 = time.perf_counter()
        r0 = O.tree_pass(self.model0, self.tok, tree, 0, self.kc0, self.kc0.copy())
        if WORKLOAD["mode"] == "typical":
            O.evaluate_posterior(r0["logits"].astype(np.float32), self.tok, tree, mode=O.TYPICAL, tau=WORKLOAD["temperature"],
                                 eps=WORKLOAD["eps"], delta=WORKLOAD["delta"])
        else:
            O.evaluate_posterior(r0["logits"].astype(np.float32), self.tok, tree, mode=O.GREEDY)
        t_lm = time.perf_counter() - t0
        t0 = time.perf_counter()
        O.tree_pass(self.model, self.tok, tree, self.L, self.kc, self.vc, want_logits=False)
        t_layers = time.perf_counter() - t0
        full = t_heads + t_lm + t_layers * self.cfg_full["n_layers"] / self.n
        desc = ("oracle, bf16 weights widened on the fly: Medusa heads + top-k (%.2fs) and LM head + acceptance (%.2fs) "
                "in full, %d of %d decoder layers at T=64, L=%d (%.2fs), layer time scaled to full depth"
                % (t_heads, t_lm, self.n, self.cfg_full["n_layers"], self.L, t_layers))
        return full, desc


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = I.model_shape(WORKLOAD["model"])
    sample = OracleSample(1, cfg, WORKLOAD["prompt"])
    times = []
    desc = ""
    for i in range(args.warmup + args.steps):
        sec, desc = sample.run()
        if i >= args.warmup:
            times.append(sec)
    sec = float(np.mean(times))
    cores = sample.cores
    value = 1.0 / sec  # random-init heads: one token per step (the root) is what the oracle accepts too
    line = {
        "metric": WORKLOAD["metric"], "value": value, "unit": "tokens/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "impl": "reference",
        # each timed step runs 1 of the identical decoder layers; ms_per_step is that sample scaled to the full depth,
        # so steps x ms_per_step exceeds the wall time of this run by design
        "extrapolated": True, "layers_run_per_step": 1, "layers_total": cfg["n_layers"],
        "config": {"workload": WORKLOAD["name"], "tree_nodes": tree_spec(WORKLOAD["tree"])["n_nodes"], "prompt": WORKLOAD["prompt"], "L_max": WORKLOAD["L_max"]},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------- GPU arm

def measure_read_peak(torch, B, stream, gib: float = 4.0, reps: int = 5):
    """Read-only DRAM bandwidth of this GPU, GB/s: one pass of 16-byte streaming loads over a buffer far larger than
    the L2, best of `reps`, CUDA events on the stream the kernel runs on."""
    n = int(gib * (1 << 30))
    buf = torch.empty(n, dtype=torch.uint8, device="cuda")
    buf.random_(0, 255)
    sink = torch.zeros(4096, dtype=torch.float32, device="cuda")
    best = 0.0
    for i in range(reps + 2):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        B.stream_read(buf, n, sink, stream.cuda_stream)
        b.record(stream)
        b.synchronize()
        if i >= 2:
            best = max(best, n / (a.elapsed_time(b) * 1e-3) / 1e9)
    del buf
    return best


def run_gpu(args):
    import torch
    import torch.distributed as dist

    from paper_2401_10774_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    spec = tree_spec(WORKLOAD["tree"])
    NB = int(WORKLOAD.get("batch", 1))  # sequences stepped together
    cfg = I.model_shape(WORKLOAD["model"], max_tree_nodes=spec["n_nodes"], max_batch=NB)
    t_setup = time.perf_counter()
    w = I.make_weights(cfg, seed=WORKLOAD["weights_seed"], dtype="bf16")

    def dev(a):
        return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda().view(torch.bfloat16)

    dw = {k: dev(v) for k, v in w.items() if k != "layers"}
    dw["layers"] = [{k: dev(v) for k, v in lw.items()} for lw in w["layers"]]
    del w
    # one stream for everything that follows: the library's launches, the host-buffer copies and the timing events
    torch.cuda.synchronize()
    stream = torch.cuda.Stream(device=local)
    torch.cuda.set_stream(stream)
    ctx = B.Context(cfg, B.BF16, WORKLOAD["L_max"], device=local, stream=stream.cuda_stream)
    tree = ctx.build_tree_buffers(B.default_tree_paths(spec["per_depth_topk"], spec["n_nodes"]))
    if args.planes != 2:
        ctx.set_option(B.OPT_ACTIVATION_PLANES, args.planes)
    ctx.set_option(B.OPT_PACK_WEIGHTS, args.pack_weights)  # read by load_weights below
    ctx.load_weights(dw)
    for b in range(NB):
        ctx.select_sequence(b)
        prompt = I.make_prompt(WORKLOAD["prompt"], cfg["vocab"], WORKLOAD["prompt_seed"] + 100 * b)
        ctx.prefill(torch.from_numpy(prompt).cuda())
    ctx.select_sequence(0)
    torch.cuda.synchronize()

    def total_len():
        n = 0
        for b in range(NB):
            ctx.select_sequence(b)
            n += ctx.state()["cache_len"]
        ctx.select_sequence(0)
        return n
    t_setup = time.perf_counter() - t_setup
    typical = WORKLOAD["mode"] == "typical"
    if typical:
        params = B.AcceptParams(mode=B.TYPICAL, temperature=WORKLOAD["temperature"], eps=WORKLOAD["eps"], delta=WORKLOAD["delta"])
    else:
        params = B.AcceptParams(mode=B.GREEDY)
    W = tree["depth"] + 1
    pinned = torch.zeros(NB * (W + 1), dtype=torch.int32).pin_memory()
    emitted_ptr, n_ptr = pinned.data_ptr(), pinned.data_ptr() + 4 * W * NB
    # typical acceptance samples the next root with Gumbel noise the caller supplies: one float [V] row per step
    n_prof = min(args.steps, 5)
    n_noise = 2 * args.warmup + 3 * args.steps + n_prof
    noise_host = noise_dev = noise_stage = None
    if typical:
        noise_host = torch.from_numpy(I.gumbel_noise(n_noise, cfg["vocab"], WORKLOAD["noise_seed"])).pin_memory()
        noise_dev = noise_host.cuda()
        noise_stage = torch.empty(cfg["vocab"], dtype=torch.float32, device="cuda")
    step_no = [0]

    def step_device_only():
        i = step_no[0]
        step_no[0] += 1
        if NB > 1:
            ctx.decode_step_batch(params, None, 1 << 30, None, None)
        else:
            ctx.decode_step(params, noise_dev[i] if typical else None, 1 << 30, None, None)

    def step_e2e():
        # what a caller does: hand the step its host-side input (the noise row, if the mode draws one), run it,
        # read the emitted tokens back on the host before deciding to go on
        i = step_no[0]
        step_no[0] += 1
        if typical:
            noise_stage.copy_(noise_host[i], non_blocking=True)
        if NB > 1:
            ctx.decode_step_batch(params, None, 1 << 30, emitted_ptr, n_ptr)
            torch.cuda.synchronize()
            return int(pinned[W * NB:W * NB + NB].sum())
        ctx.decode_step(params, noise_stage if typical else None, 1 << 30, emitted_ptr, n_ptr)
        torch.cuda.synchronize()
        return int(pinned[W])

    # both call signatures warm up (the library captures each into its own whole-step CUDA graph on second use)
    for _ in range(args.warmup):
        step_e2e()
    for _ in range(args.warmup):
        step_device_only()
    read_peak_gbs = measure_read_peak(torch, B, stream)
    L0 = total_len()
    ctx.get_profile(reset=True)
    sampler = ClockSampler(local)
    sampler.start()
    # ---- timed region 1: K steps, everything resident in HBM
    barrier()
    t_load0 = time.time()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step_device_only()
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    prof = ctx.get_profile(reset=True)
    launches = sum(v["launches"] for v in prof.values())
    L1 = total_len()
    tokens = L1 - L0
    # ---- timed region 2: the same K steps through the host-buffer call, tokens read back every step
    barrier()
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2.record()
    tokens_e2e = 0
    for _ in range(args.steps):
        tokens_e2e += step_e2e()
    e3.record()
    barrier()
    ms_e2e = e2.elapsed_time(e3)
    # ---- per-step distribution: the same K steps with an event after every step
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    evs[0].record()
    for i in range(args.steps):
        step_device_only()
        evs[i + 1].record()
    barrier()
    t_load1 = time.time()
    # the clock samples cover the three regions above (the GPU runs decode steps back to back throughout)
    clocks = sampler.stop(t_load0, t_load1)
    per_step_us = np.array([evs[i].elapsed_time(evs[i + 1]) * 1e3 for i in range(args.steps)])
    # ---- instrumented region: the same steps with CUDA events around every launch (per-kernel durations)
    ctx.get_profile(reset=True)
    ctx.set_profiling(True)
    for _ in range(n_prof):
        step_device_only()
    prof_t = ctx.get_profile(reset=True)
    ctx.set_profiling(False)
    L_end = total_len() // NB
    status = ctx.device_status()
    if status != 0:
        raise SystemExit("device status %d during the benchmark" % status)

    from paper_2401_10774_b200 import replicas

    # replicas only: the slowest rank's time, all ranks' tokens
    (ms, ms_e2e), (tokens, tokens_e2e) = replicas.reduce_over_ranks([ms, ms_e2e], [tokens, tokens_e2e], device="cuda")

    if rank == 0:
        peaks = measured_peaks()
        T = tree["T"]
        L_mid = (L0 + L1) // (2 * NB)
        sb = R.step_bytes(dict(cfg, depth=tree["depth"]), T, L_mid, tree["depth"])
        if NB > 1:  # the weights cross the HBM once for all sequences; caches, tree K/V and logits once per sequence
            per_seq = sb["kv_read"] + sb["tree_kv_write"] + sb["logits_write_read"] + sb["commit"]
            sb["total"] += (NB - 1) * per_seq
        ms_step = ms / args.steps
        step_gbs = sb["total"] / (ms_step * 1e-3) / 1e9
        # dominant kernel: the backbone GEMM launches (7 per layer + LM head)
        gemm = prof_t["gemm"]
        gemm_bytes_step = R.gemm_launch_bytes_per_step(cfg, T * NB)
        gemm_launches_step = gemm["launches"] / max(n_prof, 1)
        gemm_ms_step = gemm["ms"] / max(n_prof, 1)
        achieved = gemm_bytes_step / (gemm_ms_step * 1e-3) / 1e9 if gemm_ms_step > 0 else 0.0
        kernels = {k: dict(ms_per_step=v["ms"] / max(n_prof, 1), launches_per_step=v["launches"] / max(n_prof, 1))
                   for k, v in prof_t.items() if v["launches"]}
        att_bytes = NB * cfg["n_layers"] * R.attention_bytes(T, cfg["n_heads"], cfg["head_dim"], L_end, Hkv=I.kv_heads(cfg))
        if "tree_attention" in kernels and kernels["tree_attention"]["ms_per_step"] > 0:
            kernels["tree_attention"]["achieved_gbs"] = att_bytes / (kernels["tree_attention"]["ms_per_step"] * 1e-3) / 1e9
        if "heads_gemv" in kernels and kernels["heads_gemv"]["ms_per_step"] > 0:
            kernels["heads_gemv"]["achieved_gbs"] = R.heads_bytes(cfg["d"], cfg["vocab"], tree["depth"]) / (
                kernels["heads_gemv"]["ms_per_step"] * 1e-3) / 1e9
        kernels["gemm"]["achieved_gbs"] = achieved
        traffic, traffic_note = R.captured_traffic("gemm_tc_kernel", WORKLOAD["model"])
        line = {
            "metric": WORKLOAD["metric"],
            "value": tokens / (ms * 1e-3),
            "unit": "tokens/s",
            "n_gpus": world,
            "steps": args.steps,
            "warmup": args.warmup,
            "ms_per_step": ms_step,
            "step_us": ms_step * 1e3,
            "step_us_p10_p50_p90": [float(np.percentile(per_step_us, q)) for q in (10, 50, 90)],
            "accepted_tokens_per_step": tokens / (args.steps * world * NB),
            "higher_is_better": True,
            "scaling": "weak",
            "vs_baseline": None,
            "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": WORKLOAD["name"], "tree_nodes": T, "prompt": WORKLOAD["prompt"], "L_max": WORKLOAD["L_max"],
                       "cache_len_start": L0 // NB, "heads": cfg["n_medusa"], "replicas": world, "batch": NB, "activation_planes": args.planes, "packed_weights": bool(args.pack_weights),
                       "l2": "inputs larger than L2: every step streams %.1f GB of weights" % (sb["gemm_weights"] / 1e9)},
            "clocks": clocks,
            "e2e": {"value": tokens_e2e / (ms_e2e * 1e-3), "unit": "tokens/s",
                    "h2d_bytes_per_step": 4 * cfg["vocab"] if typical else 0,
                    "d2h_bytes_per_step": 4 * (W + 1) * NB, "ms_per_step": ms_e2e / args.steps,
                    "note": "per step: C-ABI decode_step with pinned host output buffers, stream synchronised and the "
                            "emitted tokens read on the host; " + (
                                "the step's Gumbel noise row is copied from pinned host memory first" if typical else
                                "the step takes no per-step host input in greedy mode")},
            "gpu_launches": launches,
            "step_graphs": dict(ctx.step_graph_info(), note="kernel launches replayed from whole-step CUDA graphs the "
                                                            "library captured; gpu_launches counts the kernels inside them"),
            "step_roofline": {"bytes_per_step": sb["total"], "achieved_gbs": step_gbs, "frac_of_measured": step_gbs / peaks["hbm_gbs"],
                              "frac_of_read_peak": step_gbs / read_peak_gbs if read_peak_gbs else None,
                              "frac_of_8tbs_nominal": step_gbs / 8000.0, "peak_source": peaks["source"]},
            "read_peak": {"gbs": read_peak_gbs, "how": "16-byte streaming loads over 4 GiB, nothing written, best of 5, CUDA "
                                                       "events; measured in this run before the timed regions"},
            "roofline": {"kernel": "backbone GEMM (M = 64 tree tokens), %d launches per step" % round(gemm_launches_step),
                         "bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": achieved / peaks["hbm_gbs"],
                         "frac_of_read_peak": achieved / read_peak_gbs if read_peak_gbs else None,
                         "traffic": traffic, "traffic_note": traffic_note,
                         "bytes_per_step": gemm_bytes_step, "ms_per_step": gemm_ms_step, "peak_source": peaks["source"],
                         "timing": "CUDA events around every launch in an instrumented repeat of the timed steps"},
            "kernels": kernels,
            "setup_s": t_setup,
        }
        if world == 1:
            t0 = time.perf_counter()
            sample = OracleSample(WORKLOAD["oracle_layers"], cfg, L_mid)
            sec, desc = sample.run()
            if NB > 1:
                desc += "; one sequence timed, the oracle steps the %d sequences one after the other: time x %d" % (NB, NB)
            line["cpu_baseline"] = {"value": 1.0 / sec, "unit": "tokens/s", "cores": sample.cores, "kind": "oracle", "sample": desc,
                                    "seconds_per_step": sec * NB, "wall_s": time.perf_counter() - t0}
        print(json.dumps(line))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def spawn_replicas(n: int) -> int:
    """`bench.py --gpus N` started without a launcher: start the N single-GPU replicas ourselves (one process per GPU,
    rendezvous on 127.0.0.1) and pass their exit code on."""
    import socket

    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n), "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="7b", choices=sorted(WORKLOADS), help="7b: the headline configuration")
    ap.add_argument("--pack-weights", type=int, default=1, choices=(0, 1),
                    help="1 (the library's default): the context streams its own tile-by-tile copy of the backbone matrices; "
                         "0: the row-major tensors as given")
    ap.add_argument("--planes", type=int, default=2, choices=(1, 2),
                    help="activation planes the projections read (2: hi + lo, the default and the headline; 1: hi only)")
    args = ap.parse_args()
    global WORKLOAD
    WORKLOAD = WORKLOADS[args.workload]
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.gpus < 1:
        raise SystemExit("--gpus must be >= 1")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_replicas(args.gpus))
    if world != args.gpus:
        raise SystemExit("--gpus %d does not match the launcher's WORLD_SIZE=%d" % (args.gpus, world))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
