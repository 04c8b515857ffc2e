"""The workspace-free LAMB entry point against the regular one.

ws_lamb_update_static_scratch serves callers that cannot obtain device memory
when the update runs (an optimizer plug-in under a framework that already owns
the whole GPU, a step loop that must not enter the CUDA allocator).  It must
give the same weights, moments, gathered copy and trust ratios as
ws_shard_update with a caller workspace - here checked bit for bit, on two
consecutive steps, because both calls share the library's one scratch array
and the second call finds the first call's leftovers in it.

This file sorts last on purpose, so that a run that stops at the first failure
has already run every other test."""
import ctypes as C

import pytest
import torch

from oracle import ws_oracle as O
from paper_2004_13336_b200 import binding as B
from paper_2004_13336_b200 import workloads as W
from tests._util import TOL_BF16, TOL_LAMB, bf16_to_f64, err, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda"
SHAPES = [(1,), (7,), (3, 3, 16, 32), (64, 128), (1031,), (4099, 3), (300, 301), (32,)]


def _setup(R, seed, gdtype=torch.float32):
    wl = W.Workload("t", list(SHAPES), R=R, opt="lamb", hyper={}, grad_dtype=gdtype, grad_std=1e-2, seed=seed)
    plan = B.Plan(SHAPES, R, 32)
    state = []
    for lst in W.make_state(wl, DEV):
        buf = torch.empty(plan.G, device=DEV)
        B.ws_pack(plan, lst, buf)
        state.append(buf)
    return wl, plan, state


def _grads(wl, plan, seed):
    wl.seed = seed
    out = []
    for gk in W.make_grads(wl, DEV):
        b = torch.empty(plan.G, dtype=wl.grad_dtype, device=DEV)
        B.ws_pack(plan, gk, b)
        out.append(b)
    return out


@pytest.mark.parametrize("R,gdtype", [(4, torch.float32), (7, torch.bfloat16)])
def test_static_scratch_lamb_equals_workspace_lamb_on_two_steps(R, gdtype):
    wl, plan, (w, m, v) = _setup(R, seed=21, gdtype=gdtype)
    assert plan.workspace_bytes("lamb") <= B.lib().ws_static_scratch_bytes()
    ref = [w.clone(), m.clone(), v.clone()]
    # ... and, directly, against the CPU oracle's sharded route on the same packed buffers
    oplan = O.Plan(wl.numels, R, 32)
    ow, om, ov = to_np(w), to_np(m), to_np(v)
    ws = torch.zeros(plan.workspace_bytes("lamb"), dtype=torch.uint8, device=DEV)
    for step in (1, 2):
        hd = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-6, weight_decay=0.01, momentum=0.0, grad_scale=1.0,
                  step=step)
        hy = B.make_hyper("lamb", hd)
        pg = _grads(wl, plan, seed=100 + step)          # fresh gradients every step
        og, _, _ = O.sharded_update(O.make_hyper("lamb", hd), oplan, [to_np(b) for b in pg], ow, om, ov, O.BF16)
        g_ref = torch.zeros(plan.G, dtype=torch.bfloat16, device=DEV)
        g_new = torch.zeros_like(g_ref)
        B.ws_shard_update(plan, -1, pg, ref[0], ref[1], ref[2], hy, g_ref, ws)
        B.ws_lamb_update_static_scratch(plan, pg, w, m, v, hy, g_new)
        torch.cuda.synchronize()
        assert torch.equal(w, ref[0]) and torch.equal(m, ref[1]) and torch.equal(v, ref[2]), f"step {step}"
        assert torch.equal(g_new, g_ref), f"step {step}"
        assert bool(torch.isfinite(w).all())
        for name, got, exp in (("w", w, ow), ("m", m, om), ("v", v, ov)):
            for t, (a, b) in enumerate(zip(O.unpack(oplan, to_np(got)), O.unpack(oplan, exp))):
                assert err(a, b) <= TOL_LAMB, f"step {step} {name}[{t}]"
        for a, b in zip(O.unpack(oplan, to_np(g_new)), O.unpack(oplan, og)):
            assert err(bf16_to_f64(a), bf16_to_f64(b)) <= TOL_BF16, f"step {step} gathered"


def test_static_scratch_rejects_plans_beyond_its_size():
    # 4 MiB of scratch cannot hold the partial sums of this plan: refused, nothing launched
    plan = B.Plan([(32768, 32768)] * 2, 16, 32, 2048, upload=False)      # 2.1e9 parameters, 2048-element tiles
    assert plan.workspace_bytes("lamb") > B.lib().ws_static_scratch_bytes()
    buf = torch.zeros(8, device=DEV)
    ptrs = (C.c_void_p * 16)(*([buf.data_ptr()] * 16))
    g = B.ws_grads(C.cast(ptrs, C.POINTER(C.c_void_p)), 16, 0, 0)
    s = B.ws_state(buf.data_ptr(), buf.data_ptr(), buf.data_ptr())
    hy = B.make_hyper("lamb", W.bert_large().hyper)
    rc = B.lib().ws_lamb_update_static_scratch(plan.handle, C.byref(g), C.byref(s), C.byref(hy), None, None)
    assert rc == 7
    assert B.lib().ws_status_string(rc) == b"size beyond a fixed limit"
    hy_adam = B.make_hyper("adam", W.tiny().hyper)
    assert B.lib().ws_lamb_update_static_scratch(plan.handle, C.byref(g), C.byref(s), C.byref(hy_adam), None, None) == 1
    torch.cuda.synchronize()
    assert float(buf.sum()) == 0.0
