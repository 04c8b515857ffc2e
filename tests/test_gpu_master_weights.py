"""Fused formatting with the fp32 weight tensors as the master copy (paper Section 5.1: the formatting
is fused into the reduce-scatter and the all-gather, padding in place).  ws_fused_update with
state->w == NULL reads each weight from its tensor and writes it back there: no sharded copy of w
exists and the updated weight is written exactly once.  Checked against the oracle's plain unsharded
definition and, bit for bit, against the form that keeps a sharded w."""
import numpy as np
import pytest
import torch

from oracle import ws_oracle as O
from paper_2004_13336_b200 import binding as B
from paper_2004_13336_b200 import workloads as W
from tests._util import TOL_FP32, TOL_LAMB, err, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda"
SHAPES = [(1,), (7,), (3, 3, 16, 32), (64, 128), (1031,), (5, 1, 9), (4099, 3), (300, 301), (32,), (20011,), (0,)]

HYPER = {
    "sgdm": dict(lr=0.1, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=5e-5, momentum=0.9, grad_scale=1.0, step=10),
    "adam": dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0, momentum=0.0, grad_scale=1.0, step=10),
    "lamb": dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-6, weight_decay=0.01, momentum=0.0, grad_scale=1.0, step=10),
    "lars": dict(lr=10.0, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=5e-5, momentum=0.9, grad_scale=1.0, step=10,
                 trust_coeff=0.001),
}


def _guarded_views(numels, fill, misalign):
    """One big buffer per tensor with guard zones; views start 32- (or only 16-) byte aligned."""
    bigs, views = [], []
    for n in numels:
        big = torch.full((n + 160,), fill, dtype=torch.float32, device=DEV)
        start = 64 + (4 if misalign else 0)
        bigs.append(big)
        views.append(big[start:start + n])
    return bigs, views


@pytest.mark.parametrize("opt", ["sgdm", "adam", "lamb", "lars"])
@pytest.mark.parametrize("R", [1, 3, 8, 40])
@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("layout,misalign", [("per_tensor", False), ("concat", False), ("per_tensor", True)])
def test_weight_tensors_as_master_copy(opt, R, gdtype, layout, misalign):
    wl = W.Workload("t", list(SHAPES), R=R, opt=opt, hyper={}, grad_dtype=gdtype, grad_std=1e-2, seed=R + 7)
    w, m, v = W.make_state(wl, DEV)
    g = W.make_grads(wl, DEV)
    numels = wl.numels
    plan = B.Plan(SHAPES, R, 32, layout=layout)
    hy = B.make_hyper(opt, HYPER[opt])
    has_v = opt in ("adam", "lamb")
    # oracle: the plain definition on whole tensors
    hs = O.make_hyper(opt, HYPER[opt])
    ow, om, ov = [to_np(x) for x in w], [to_np(x) for x in m], [to_np(x) for x in v]
    orho = O.update_unsharded(hs, [[to_np(x) for x in gk] for gk in g], ow, om, ov if has_v else None)
    # the form with a sharded copy of w (reference for bit equality)
    pm, pv, pw = (torch.empty(plan.G, device=DEV) for _ in range(3))
    B.ws_pack(plan, w, pw); B.ws_pack(plan, m, pm); B.ws_pack(plan, v, pv)
    rm, rv = pm.clone(), pv.clone()
    gt = B.TensorTable(plan, g)
    ref_out = [torch.zeros_like(x) for x in w]
    ws = torch.zeros(max(32, plan.workspace_bytes(opt)), dtype=torch.uint8, device=DEV)
    B.ws_fused_update(plan, -1, gt, pw, rm, rv if has_v else None, hy, B.TensorTable(plan, [ref_out]), ws)
    # master form: the weight tensors hold w before the call and w' after it
    bigs, views = _guarded_views(numels, 7.0, misalign)
    for dst, src in zip(views, w):
        dst.copy_(src)
    ws2 = torch.zeros_like(ws)
    B.ws_fused_update(plan, -1, gt, None, pm, pv if has_v else None, hy, B.TensorTable(plan, [views]), ws2)
    torch.cuda.synchronize()
    tol = TOL_FP32 if opt in ("sgdm", "adam") else TOL_LAMB
    for t, (a, b) in enumerate(zip(views, ow)):
        assert err(to_np(a), b) <= tol, f"w[{t}]"
    # 16-byte-only alignment runs the 128-bit variant: the norm partial sums are grouped differently
    exact = not (misalign and opt in ("lamb", "lars"))
    for a, b in zip(views, ref_out):
        if exact:
            assert torch.equal(a, b)
        else:
            assert err(to_np(a), to_np(b)) <= 2e-7
    if exact or opt == "lamb":                 # (LARS folds the local rate into its momentum)
        assert torch.equal(pm, rm)
    else:
        assert err(to_np(pm), to_np(rm)) <= 2e-7
    if has_v:
        assert torch.equal(pv, rv)
    for big, n in zip(bigs, numels):           # nothing outside the tensors was written
        start = 64 + (4 if misalign else 0)
        assert bool((big[:start] == 7.0).all()) and bool((big[start + n:] == 7.0).all())
    if opt in ("lamb", "lars"):
        got = B.lamb_ratios(plan, ws2).cpu().numpy().astype(np.float64)
        for t, n in enumerate(numels):
            if n:
                assert abs(got[t] / orho[t] - 1.0) <= TOL_LAMB


def test_master_copy_shard_by_shard_and_argument_checks():
    R = 5
    wl = W.Workload("t", list(SHAPES), R=R, opt="adam", hyper={}, grad_std=1e-2, seed=3)
    w, m, v = W.make_state(wl, DEV)
    g = W.make_grads(wl, DEV)
    plan = B.Plan(SHAPES, R, 32)
    hy = B.make_hyper("adam", HYPER["adam"])
    pm, pv = torch.empty(plan.G, device=DEV), torch.empty(plan.G, device=DEV)
    B.ws_pack(plan, m, pm); B.ws_pack(plan, v, pv)
    am, av = pm.clone(), pv.clone()
    gt = B.TensorTable(plan, g)
    w_all = [x.clone() for x in w]
    w_one = [x.clone() for x in w]
    B.ws_fused_update(plan, -1, gt, None, am, av, hy, B.TensorTable(plan, [w_all]))
    wt = B.TensorTable(plan, [w_one])
    S = plan.S
    for r in range(R):                         # one replica's slice at a time
        sl = slice(r * S, (r + 1) * S)
        B.ws_fused_update(plan, r, gt, None, pm[sl], pv[sl], hy, wt)
    assert torch.equal(am, pm) and torch.equal(av, pv)
    for a, b in zip(w_all, w_one):
        assert torch.equal(a, b)
    # bf16 weight tensors cannot be the master copy; nor can several weight lists
    wb = [x.to(torch.bfloat16) for x in w]
    with pytest.raises(B.WsError) as e:
        B.ws_fused_update(plan, -1, gt, None, pm, pv, hy, B.TensorTable(plan, [wb]))
    assert e.value.status == 1
    with pytest.raises(B.WsError) as e:
        B.ws_fused_update(plan, -1, gt, None, pm, pv, hy, B.TensorTable(plan, [w_all, w_one]))
    assert e.value.status == 1
    # the packed-buffer route always needs its sharded w
    with pytest.raises(B.WsError) as e:
        B.ws_shard_update(plan, -1, [torch.zeros(plan.G, device=DEV)] * R, None, pm, pv, hy)
    assert e.value.status == 1


def test_master_copy_adafactor_matches_the_sharded_form():
    shapes = [(7,), (64, 128), (4099, 3), (300, 301), (2, 9001), (24, 2048), (3, 8192)]
    R = 4
    wl = W.Workload("t", list(shapes), R=R, opt="adafactor", hyper={}, grad_std=1e-2, seed=11)
    w, _, _ = W.make_state(wl, DEV)
    g = W.make_grads(wl, DEV)
    plan = B.Plan(shapes, R, 32)
    h = dict(lr=1e-2, beta1=0.0, beta2=0.0, eps=1e-30, weight_decay=0.0, momentum=0.0, grad_scale=1.0, step=10,
             eps2=1e-3, clip_threshold=1.0, decay_exponent=0.8)
    hy = B.make_hyper("adafactor", h)
    f0 = W.make_factored_state(wl, plan.factored_elems, DEV)
    fa, fb = f0.clone(), f0.clone()
    pw = torch.empty(plan.G, device=DEV)
    B.ws_pack(plan, w, pw)
    gt = B.TensorTable(plan, g)
    ref_out = [torch.zeros_like(x) for x in w]
    ws = torch.zeros(plan.workspace_bytes("adafactor"), dtype=torch.uint8, device=DEV)
    B.ws_fused_update(plan, -1, gt, pw, None, fa, hy, B.TensorTable(plan, [ref_out]), ws)
    wm = [x.clone() for x in w]
    ws2 = torch.zeros_like(ws)
    B.ws_fused_update(plan, -1, gt, None, None, fb, hy, B.TensorTable(plan, [wm]), ws2)
    torch.cuda.synchronize()
    # (the row / column sums are formed with floating-point atomic adds: equal to rounding, not bit for bit)
    for a, b in zip(wm, ref_out):
        assert err(to_np(a), to_np(b)) <= 1e-6
    assert err(to_np(fb), to_np(fa)) <= 1e-5
