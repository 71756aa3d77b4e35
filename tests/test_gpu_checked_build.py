"""The checked flavour of the library (-DMEDUSA_DEBUG_CHECKS): the same entry points plus validation kernels after the
stages of a step, which record MEDUSA_ERR_NONFINITE / MEDUSA_ERR_BOUNDS in the device status word.  It stands in for
a memory checker where none can be run: nothing traps, nothing is skipped, results equal the default library's.

A process can hold one flavour, so the checked library runs in a child process and reports as JSON.
"""
import json
import os
import subprocess
import sys

import numpy as np
import pytest

from paper_2401_10774_b200 import inputs as I

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import json, sys
import numpy as np, torch
from paper_2401_10774_b200 import binding as B, inputs as I
if sys.argv[1] == "checked":
    B.use_checked_library()
out = dict(checks=int(B.lib().medusa_debug_checks_enabled()))
cfg = I.model_shape("tiny")
spec = I.TREE_SPECS["dense22"]

def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()

def ctx_with(w):
    ctx = B.Context(cfg, B.F32, 128)
    ctx.build_tree_buffers(B.default_tree_paths(spec["per_depth_topk"], spec["n_nodes"]))
    dw = {k: dev(v) for k, v in w.items() if k != "layers"}
    dw["layers"] = [{k: dev(v) for k, v in lw.items()} for lw in w["layers"]]
    ctx.load_weights(dw)
    return ctx

w = I.make_weights(cfg, seed=0, dtype="f32", head_init="lm_copy")
prompt = I.make_prompt(32, cfg["vocab"], 1)
# 1. a clean run: status stays 0, tokens as the default library gives them
ctx = ctx_with(w)
got = ctx.generate(prompt, 24, B.AcceptParams(mode=B.GREEDY))
out["tokens"] = got["tokens"].tolist()
out["status_clean"] = ctx.device_status()
# 2. a token outside the vocabulary in a tree pass: recorded, nothing faults (the embedding clamps the index)
tok = torch.full((7,), cfg["vocab"] + 5, dtype=torch.int32, device="cuda")
ctx.tree_pass(tok)
try:
    out["status_bad_token"] = ctx.device_status()
except B.MedusaError as e:
    out["status_bad_token"] = e.code
ctx.reset()
out["status_after_reset"] = ctx.device_status()
# 3. a cache length beyond the cache in the stand-alone attention: recorded, the kernel clamps it
H, D, T = cfg["n_heads"], cfg["head_dim"], 7
q = torch.zeros(T, H, D, device="cuda"); kn = torch.zeros_like(q); vn = torch.zeros_like(q)
kc = torch.zeros(H, 128, D, device="cuda"); vc = torch.zeros_like(kc); o = torch.zeros_like(q)
ctx.tree_attention(q, kn, vn, kc, vc, torch.tensor([4000], dtype=torch.int32, device="cuda"), False, o)
try:
    out["status_bad_len"] = ctx.device_status()
except B.MedusaError as e:
    out["status_bad_len"] = e.code
ctx.close()
# 4. a NaN in the LM head: the backbone logits of the first pass are not finite
w2 = dict(w); w2["lm_head"] = w["lm_head"].copy(); w2["lm_head"][3, 5] = np.nan
ctx = ctx_with(w2)
ctx.prefill(dev(prompt))
try:
    out["status_nan"] = ctx.device_status()
except B.MedusaError as e:
    out["status_nan"] = e.code
ctx.close()
print("RESULT " + json.dumps(out))
"""


def _run(flavour):
    env = dict(os.environ, PYTHONPATH=ROOT + os.pathsep + os.environ.get("PYTHONPATH", ""))
    r = subprocess.run([sys.executable, "-c", CHILD, flavour], capture_output=True, text=True, cwd=ROOT, env=env, timeout=600)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    line = [l for l in r.stdout.splitlines() if l.startswith("RESULT ")][-1]
    return json.loads(line[len("RESULT "):])


def test_checked_library_records_what_the_default_library_lets_pass():
    NONFINITE, BOUNDS = -8, -9
    from paper_2401_10774_b200 import build as lib_build
    lib_build.build_library(debug_checks=True)  # a no-op when the checked flavour is already up to date
    checked = _run("checked")
    plain = _run("default")
    assert checked["checks"] == 1 and plain["checks"] == 0
    assert checked["tokens"] == plain["tokens"], "the validation kernels must not change any result"
    assert checked["status_clean"] == 0 and plain["status_clean"] == 0
    assert checked["status_bad_token"] == BOUNDS and checked["status_after_reset"] == 0
    assert checked["status_bad_len"] == BOUNDS
    assert checked["status_nan"] == NONFINITE
    # the default library computes the same things without looking
    assert plain["status_bad_token"] == 0 and plain["status_bad_len"] == 0 and plain["status_nan"] == 0
