"""CPU-only checks of the host side: the C-ABI library loads and exports what the header declares, the host
tree builder agrees bit for bit with the oracle, argument validation, the byte accounting against the paper's
printed operational intensities, and the replica aggregation over a 2-rank gloo group."""
import ctypes as C
import json
import os
import re

import numpy as np
import pytest

from paper_2401_10774_b200 import binding as B
from paper_2401_10774_b200 import inputs as I
from paper_2401_10774_b200 import roofline as R

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "medusa.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = sorted(set(re.findall(r"\b(medusa_[a-z_0-9]+)\s*\(", hdr)))
    assert {"medusa_heads", "medusa_build_tree_buffers", "medusa_tree_attention", "medusa_evaluate_posterior",
            "medusa_accept_and_update_kv", "medusa_decode_step"} <= set(names)
    lib = B.lib()
    for n in names:
        assert hasattr(lib, n), "library does not export %s" % n


def test_binding_structs_mirror_the_header():
    # the ctypes mirror of medusa_model_desc lists the header's fields in the header's order (all 4 bytes wide)
    hdr = open(os.path.join(ROOT, "include", "medusa.h")).read()
    body = re.search(r"typedef struct \{(.*?)\} medusa_model_desc;", hdr, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = []
    for decl in body.split(";"):
        m = re.match(r"\s*(int32_t|float)\s+(.*)", decl.strip(), flags=re.S)
        if m:
            fields += [(n.strip(), m.group(1)) for n in m.group(2).split(",")]
    got = [(n, "float" if t is B.C.c_float else "int32_t") for n, t in B.ModelDesc._fields_]
    assert got == fields
    assert B.C.sizeof(B.ModelDesc) == 4 * len(fields)
    assert "n_kv_heads" in dict(fields)


def test_shapes_with_unequal_key_value_heads_are_validated():
    # every key/value head must serve the same number of query heads: checked before any device is touched
    bad = dict(I.model_shape("tiny"), n_kv_heads=3)  # 4 query heads
    with pytest.raises(B.MedusaError) as e:
        B.Context(bad, B.F32, 64)
    assert e.value.code == B.ERR_SHAPE
    assert I.kv_heads(I.model_shape("mistral7b")) == 8 and I.kv_heads(I.model_shape("7b")) == 32


def test_create_fails_loudly_without_a_device():
    import torch

    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises(B.MedusaError) as e:
        B.Context(I.model_shape("tiny"), B.F32, 64)
    assert e.value.code == B.ERR_CUDA


@pytest.mark.parametrize("name", sorted(I.TREE_SPECS))
def test_host_tree_buffers_bit_exact_vs_oracle(oracle, name):
    spec = I.TREE_SPECS[name]
    p_lib = B.default_tree_paths(spec["per_depth_topk"], spec["n_nodes"])
    p_ora = oracle.default_tree_paths(spec["per_depth_topk"], spec["n_nodes"])
    assert {tuple(r) for r in p_lib.tolist()} == {tuple(r) for r in p_ora.tolist()}
    # each side builds from the OTHER side's path list as well (order of the input rows must not matter)
    for paths in (p_lib, p_ora[::-1]):
        t_lib, t_ora = B.build_tree_buffers(None, paths), oracle.build_tree_buffers(paths)
        for k in ("T", "P", "depth", "topk"):
            assert t_lib[k] == t_ora[k]
        for k in ("mask", "pos", "tree_idx", "parent", "retrieve"):
            assert np.array_equal(t_lib[k], t_ora[k]), k


@pytest.mark.parametrize("topk,n_nodes", [((6, 4, 3, 2, 2), 128), ((10, 6, 4, 3, 2), 256)])
def test_host_large_tree_buffers_bit_exact_vs_oracle(oracle, topk, n_nodes):
    # trees of more than 64 nodes (Sec. 3.3.1, Fig. 4): masks of several 64-bit words per node
    p_lib, p_ora = B.default_tree_paths(topk, n_nodes), oracle.default_tree_paths(topk, n_nodes)
    assert {tuple(r) for r in p_lib.tolist()} == {tuple(r) for r in p_ora.tolist()}
    t_lib, t_ora = B.build_tree_buffers(None, p_lib), oracle.build_tree_buffers(p_ora[::-1])
    assert t_lib["mask"].shape == (n_nodes, (n_nodes + 63) // 64)
    for k in ("T", "P", "depth", "topk"):
        assert t_lib[k] == t_ora[k]
    for k in ("mask", "pos", "tree_idx", "parent", "retrieve"):
        assert np.array_equal(t_lib[k], t_ora[k]), k


def test_host_tree_random_prefix_closed_trees(oracle):
    g = I.rng(17, "random-trees")
    for trial in range(40):
        depth = int(g.integers(1, 6))
        nodes = {()}
        target = int(g.integers(1, 64)) if trial % 3 else int(g.integers(65, 257))  # a third of them: multi-word masks
        for _ in range(8000):
            if len(nodes) >= target:
                break
            par = sorted(nodes)[int(g.integers(0, len(nodes)))]
            if len(par) < depth:
                nodes.add(par + (int(g.integers(0, 5)),))
        rows = [list(n) + [-1] * (depth - len(n)) for n in nodes if n]
        if not rows:
            continue
        paths = np.array(rows, dtype=np.int32)
        g.shuffle(paths)
        t_lib, t_ora = B.build_tree_buffers(None, paths), oracle.build_tree_buffers(paths)
        for k in ("mask", "pos", "tree_idx", "parent", "retrieve"):
            assert np.array_equal(t_lib[k], t_ora[k]), (trial, k)
    # root-only tree (plain decoding)
    t = B.build_tree_buffers(None, np.zeros((0, 1), dtype=np.int32))
    assert (t["T"], t["P"], t["depth"], t["topk"]) == (1, 1, 0, 0) and t["retrieve"].tolist() == [[0]]


def test_tree_from_accuracies_bit_exact_vs_oracle(oracle):
    """The library's best-first construction (Sec. 2.3.3) adds the same nodes in the same order as the oracle's
    literal greedy scan, on calibration-like tables, tables with exact ties and zero entries, and at the size limit."""
    g = I.rng(23, "accuracy-tables")
    cases = []
    for trial in range(30):
        depth, topk = int(g.integers(1, 6)), int(g.integers(1, 8))
        acc = np.sort(g.random((depth, topk)), axis=1)[:, ::-1] * np.linspace(0.95, 0.35, depth)[:, None]
        if trial % 3 == 1:
            acc = np.round(acc * 4) / 4      # many exact ties, some zeros and ones
        if trial % 3 == 2:
            g.shuffle(acc, axis=1)           # rows need not be sorted by rank
        total = sum(topk ** k for k in range(1, depth + 1))
        cases.append((np.ascontiguousarray(acc), int(min(256, 1 + total, g.integers(2, 257 if len(cases) % 2 else 65)))))
    cases.append((np.array([[1 / (i + 1) for i in range(10)]] * 4), 64))
    for acc, n_nodes in cases:
        p_lib, e_lib = B.tree_paths_from_accuracies(acc, n_nodes)
        p_ora, e_ora = oracle.tree_paths_from_accuracies(acc, n_nodes)
        assert np.array_equal(p_lib, p_ora), (acc.shape, n_nodes)
        assert e_lib == e_ora
        t = B.build_tree_buffers(None, p_lib)   # prefix-closed, distinct: accepted by the tree builder
        assert t["T"] == n_nodes
    # the surrogate table reproduces the default 64-node tree of the benchmark configuration
    spec = I.TREE_SPECS["sparse64_d4"]
    acc = np.zeros((4, 4))
    for k, s_k in enumerate(spec["per_depth_topk"]):
        acc[k, :s_k] = [1.0 / (i + 1) for i in range(s_k)]
    p, _ = B.tree_paths_from_accuracies(acc, spec["n_nodes"])
    d = B.default_tree_paths(spec["per_depth_topk"], spec["n_nodes"])
    assert {tuple(r) for r in p.tolist()} == {tuple(r) for r in d.tolist()}
    for bad, n in ((np.array([[1.5]]), 2), (np.array([[float("nan")]]), 2), (np.array([[0.5, 0.1]]), 4),
                   (np.full((2, 16), 0.5), 258)):
        with pytest.raises(B.MedusaError) as e:
            B.tree_paths_from_accuracies(bad, n)
        assert e.value.code in (B.ERR_INVALID_ARG, B.ERR_SHAPE)


def test_host_tree_rejects_invalid_input():
    bad = [np.array([[0, 0]]), np.array([[0, -1], [0, -1]]), np.array([[-1, 0]]), np.array([[-1, -1]])]
    for p in bad:
        with pytest.raises(B.MedusaError) as e:
            B.build_tree_buffers(None, p.astype(np.int32))
        assert e.value.code == B.ERR_INVALID_ARG
    too_many = np.array([[i] for i in range(256)], dtype=np.int32)  # 257 nodes
    with pytest.raises(B.MedusaError) as e:
        B.build_tree_buffers(None, too_many)
    assert e.value.code == B.ERR_SHAPE
    with pytest.raises(B.MedusaError):
        B.default_tree_paths((2, 2), 100)  # more nodes than the Cartesian tree has


def test_byte_accounting_reproduces_the_papers_operational_intensities():
    gold = json.load(open(os.path.join(ROOT, "tests", "golden", "paper_operational_intensity.json")))
    for q, oi in gold["attention_s1024_d128"].items():
        assert abs(R.operational_intensity_attention_unfused(1024, int(q), 128) - oi) < 0.006
    for s, oi in gold["attention_q64_d128_by_seq"].items():
        assert abs(R.operational_intensity_attention_unfused(int(s), 64, 128) - oi) < 0.006
    for q, oi in gold["linear_h6656_i17920_batch1"].items():
        assert abs(R.operational_intensity_linear(int(q), 6656, 17920) - oi) < 0.006
    # the step accounting used by the benchmark: 7B, T = 64
    cfg = I.model_shape("7b")
    sb = R.step_bytes(dict(cfg, depth=4), 64, 512, 4)
    assert abs(sb["gemm_weights"] / 1e9 - 13.214) < 0.01 and abs(sb["heads"] / 1e9 - 1.183) < 0.001
    assert abs(R.attention_bytes(64, 32, 128, 1024) / 1e6 - 18.87) < 0.01
    assert abs(R.attention_bytes(64, 32, 128, 4096) / 1e6 - 69.21) < 0.01


def _replica_worker(rank, world, port, q):
    import torch.distributed as dist

    from paper_2401_10774_b200 import replicas

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    times, counts = replicas.reduce_over_ranks([10.0 + rank, 5.0 - rank], [100 + rank, 7])
    q.put((rank, times, counts))
    dist.barrier()
    dist.destroy_process_group()


def test_replica_aggregation_two_ranks_gloo():
    import torch.multiprocessing as mp

    from paper_2401_10774_b200 import replicas

    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_replica_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, times, counts in res:
        assert times == [11.0, 5.0] and counts == [201, 14]
    # whole-job throughput = all tokens over the slowest rank's time
    assert replicas.aggregate_throughput(201, 11.0) == pytest.approx(201 / 0.011)
    # without a process group the call is the identity
    assert replicas.reduce_over_ranks([3.0], [4]) == ([3.0], [4])
