"""The bounds-checking debug build (-DWS_DEBUG_BOUNDS): every kernel compares each work item's range
with the extents of its buffers and reports a violation as a bit in a status word instead of touching
memory.  The test runs in a child process (the environment variable WS_DEBUG_BOUNDS=1 makes the binding
load libws_debug.so): the self-test must raise its bit (an index outside its extent, nothing accessed),
a set of small updates on every route must leave the word at 0, and their results must equal those of
the regular library bit for bit (the checks change no arithmetic)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r'''
import hashlib, json, sys
import torch
from paper_2004_13336_b200 import binding as B, build as ws_build, workloads as W
ws_build.build(debug=B.DEBUG_BOUNDS)
L = B.lib()
out = {"enabled": int(L.ws_debug_bounds_enabled())}
if out["enabled"]:
    assert B.debug_bounds_read() == 0
    assert L.ws_debug_bounds_selftest(None) == 0
    out["selftest_bits"] = B.debug_bounds_read()
    out["after_clear"] = B.debug_bounds_read()
DEV = "cuda"
shapes = [(1,), (7,), (3, 3, 16, 32), (64, 128), (1031,), (4099, 3), (300, 301), (0,), (20011,), (512, 1024)]
digest = hashlib.sha256()
for opt, R, layout in (("sgdm", 3, "per_tensor"), ("adam", 8, "concat"), ("lamb", 8, "per_tensor"), ("lamb", 3, "concat"),
                       ("lars", 5, "per_tensor"), ("adafactor", 4, "per_tensor")):
    wl = W.Workload("t", list(shapes), R=R, opt=opt, hyper={}, grad_std=1e-2, seed=R)
    base = {"sgdm": W.resnet50, "adam": W.transformer, "lamb": W.bert_large, "lars": W.resnet50_lars,
            "adafactor": W.transformer_adafactor}[opt]().hyper
    hy = B.make_hyper(opt, base)
    w, m, v = W.make_state(wl, DEV)
    g = W.make_grads(wl, DEV)
    plan = B.Plan(shapes, R, 32, layout=layout)
    bufs = []
    for lst in (w, m, v):
        b = torch.empty(plan.G, device=DEV)
        B.ws_pack(plan, lst, b)
        bufs.append(b)
    pw, pm, pv = bufs
    if opt in ("sgdm", "lars"):
        pv = None
    if opt == "adafactor":
        pm, pv = None, W.make_factored_state(wl, plan.factored_elems, DEV)
    pg = []
    for gk in g:
        b = torch.empty(plan.G, device=DEV)
        B.ws_pack(plan, gk, b)
        pg.append(b)
    ws = torch.zeros(max(32, plan.workspace_bytes(opt)), dtype=torch.uint8, device=DEV)
    gathered = torch.zeros(plan.G, dtype=torch.bfloat16, device=DEV)
    B.ws_shard_update(plan, -1, pg, pw, pm, pv, hy, gathered, ws)                 # packed buffers, all shards
    if opt in ("sgdm", "adam") and layout == "per_tensor":
        S = plan.S
        B.ws_shard_update(plan, 1, pg, pw[S:2 * S], pm[S:2 * S], pv[S:2 * S] if pv is not None else None, hy, gathered)
    outs = [torch.zeros(n, dtype=torch.bfloat16, device=DEV) for n in wl.numels]
    B.ws_unpack(plan, gathered, outs)
    fw = [x.clone() for x in w]
    B.ws_fused_update(plan, -1, B.TensorTable(plan, g), None, pm, pv, hy, B.TensorTable(plan, [fw]), ws)   # fused, master weights
    torch.cuda.synchronize()
    if opt != "adafactor":      # (its row / column sums are floating-point atomic adds: not bit-stable)
        for t in [pw, gathered] + fw + ([pm] if pm is not None else []):
            digest.update(t.cpu().view(torch.uint8).numpy().tobytes() if t.numel() else b"")
if out["enabled"]:
    out["bits_after_updates"] = B.debug_bounds_read()
out["digest"] = digest.hexdigest()
print("RESULT " + json.dumps(out))
'''


def _run(debug: bool):
    env = dict(os.environ, PYTHONPATH=ROOT)
    env.pop("WS_DEBUG_BOUNDS", None)
    if debug:
        env["WS_DEBUG_BOUNDS"] = "1"
    r = subprocess.run([sys.executable, "-c", CHILD], env=env, capture_output=True, text=True, cwd=ROOT, timeout=1500)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]
    line = [l for l in r.stdout.splitlines() if l.startswith("RESULT ")][-1]
    return json.loads(line[len("RESULT "):])


def test_debug_build_reports_violations_as_bits_and_is_clean_on_valid_calls():
    dbg = _run(True)
    assert dbg["enabled"] == 1
    assert dbg["selftest_bits"] == 0x40000000 and dbg["after_clear"] == 0
    assert dbg["bits_after_updates"] == 0
    ref = _run(False)
    assert ref["enabled"] == 0
    assert dbg["digest"] == ref["digest"]          # the checks change no arithmetic


def test_regular_build_has_no_debug_calls():
    from paper_2004_13336_b200 import binding as B
    import ctypes as C
    if B.DEBUG_BOUNDS:
        pytest.skip("this process runs the debug build")
    assert B.lib().ws_debug_bounds_enabled() == 0
    bits = C.c_uint32(7)
    assert B.lib().ws_debug_bounds_read(C.byref(bits), 0) == 1 and bits.value == 0
    assert B.lib().ws_debug_bounds_selftest(None) == 1
