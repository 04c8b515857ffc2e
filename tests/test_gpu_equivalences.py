"""Randomised equivalences between the library's entry points, all on the GPU: the shard-by-shard
forms against the all-shard call, ws_pack_sets against ws_pack, the fused route against the
separate kernels, and one kernel per replica over R weight lists against the unpacked gathered
buffer - over random tensor lists (also more than 1024 tensors), shard counts up to 1024,
alignments, tile sizes, layouts, optimizers and dtypes.  Bit for bit, except where a shard's slices
are less aligned than the whole buffers (the norm-based optimizers then sum in another order)."""
import numpy as np
import pytest
import torch

from paper_2004_13336_b200 import binding as B
from paper_2004_13336_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda"
POOL = [0, 1, 2, 5, 8, 31, 32, 33, 100, 255, 256, 1000, 1024, 1025, 2048, 4097, 9001, 30011, 70001]


@pytest.mark.parametrize("case", range(40))
def test_entry_points_agree(case):
    rng = np.random.default_rng(9000 + case)
    big_T = case % 13 == 5
    T = int(rng.integers(1030, 1200)) if big_T else int(rng.integers(1, 16))
    numel = [int(x) for x in rng.choice(POOL[:8] if big_T else POOL, T)]
    if sum(numel) == 0:
        numel[0] = 40
    R = int(rng.choice([1, 3, 8] if big_T else [1, 2, 3, 4, 7, 8, 12, 33, 100]))
    if case % 13 == 9:
        R, numel = int(rng.choice([257, 600, 1024])), numel[:4]
        if sum(numel) == 0:
            numel[0] = 40
    shapes = [(k,) for k in numel]
    A, tile = int(rng.choice([8, 16, 32, 128])), int(rng.choice([0, 1024, 2048]))
    layout = str(rng.choice(["per_tensor", "concat"]))
    opt = str(rng.choice(["sgdm", "adam", "lamb", "lars"]))
    gdt = torch.bfloat16 if rng.random() < 0.4 else torch.float32
    odt = torch.bfloat16 if rng.random() < 0.4 else torch.float32
    wl = W.Workload("f", shapes, R=R, opt=opt, hyper={}, grad_dtype=gdt, grad_std=1e-3, seed=case)
    h = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0, momentum=0.0, grad_scale=1.0,
             step=int(rng.integers(1, 20)))
    if opt == "sgdm":
        h.update(lr=0.1, momentum=0.9, weight_decay=5e-5)
    if opt == "lamb":
        h.update(eps=1e-6, weight_decay=0.01)
    if opt == "lars":
        h.update(lr=10.0, momentum=0.9, weight_decay=5e-5, trust_coeff=0.001)
    hy = B.make_hyper(opt, h)
    w, m, v = W.make_state(wl, DEV)
    g = W.make_grads(wl, DEV)
    plan = B.Plan(shapes, R, A, tile, layout=layout)
    S, G = plan.S, plan.G
    has_v = opt in ("adam", "lamb")
    norm_based = opt in ("lamb", "lars")

    def packed(lst, dt=torch.float32):
        b = torch.full((G,), float("nan"), dtype=dt, device=DEV)
        B.ws_pack(plan, lst, b)
        return b
    pw, pm, pv = packed(w), packed(m), packed(v)
    pg = [packed(gk, gdt) for gk in g]
    bits = torch.int16 if gdt == torch.bfloat16 else torch.int32
    many = [torch.full((G,), float("nan"), dtype=gdt, device=DEV) for _ in range(R)]
    B.ws_pack_sets(plan, B.TensorTable(plan, g), many)
    for a, b in zip(pg, many):
        assert torch.equal(a.view(bits), b.view(bits)), "ws_pack_sets"

    aw, am, av = pw.clone(), pm.clone(), pv.clone()
    ws = torch.full((max(16, plan.workspace_bytes(opt)),), 0xFF, dtype=torch.uint8, device=DEV)
    ga = torch.full((G,), 5.0, dtype=odt, device=DEV)
    B.ws_shard_update(plan, -1, pg, aw, am, av if has_v else None, hy, ga, ws)
    assert bool(torch.isfinite(aw).all())

    bw, bm, bv = pw.clone(), pm.clone(), pv.clone()
    gb = torch.full((G,), 5.0, dtype=odt, device=DEV)
    ws2 = torch.full_like(ws, 0xFF)
    sm = int(rng.integers(2))
    sl = [slice(r * S, (r + 1) * S) for r in range(R)]
    gr = (lambda r: [b[sl[r]] for b in pg]) if sm else (lambda r: pg)
    if not norm_based:
        for r in range(R):
            B.ws_shard_update(plan, r, gr(r), bw[sl[r]], bm[sl[r]], bv[sl[r]] if has_v else None, hy, gb, None,
                              slice_mode=sm)
    else:
        for r in range(R):
            if opt == "lamb":
                B.ws_lamb_partial(plan, r, gr(r), bw[sl[r]], bm[sl[r]], bv[sl[r]], hy, ws2, slice_mode=sm)
            else:
                B.ws_lars_partial(plan, r, gr(r), bw[sl[r]], bm[sl[r]], hy, ws2, slice_mode=sm)
        if opt == "lamb":
            B.ws_lamb_finalize(plan, ws2)
        else:
            B.ws_lars_finalize(plan, hy, ws2)
        for r in range(R):
            if opt == "lamb":
                B.ws_lamb_apply(plan, r, bw[sl[r]], bm[sl[r]], bv[sl[r]], hy, ws2, gb)
            else:
                B.ws_lars_apply(plan, r, bw[sl[r]], bm[sl[r]], hy, ws2, gb)
    for x, y, nm in ((aw, bw, "w"), (am, bm, "m"), (av, bv, "v"), (ga, gb, "gathered")):
        if nm == "v" and not has_v:
            continue
        if norm_based:
            assert torch.allclose(x.float(), y.float(), rtol=1e-2 if nm == "gathered" else 2e-5, atol=1e-7), nm
        else:
            assert torch.equal(x, y), nm

    fw, fm, fv = pw.clone(), pm.clone(), pv.clone()
    outs = [torch.full((k,), 9.0, dtype=odt, device=DEV) for k in numel]
    B.ws_fused_update(plan, -1, B.TensorTable(plan, g), fw, fm, fv if has_v else None, hy,
                      B.TensorTable(plan, [outs]), torch.full_like(ws, 0xFF))
    ref = [torch.full((k,), 7.0, dtype=odt, device=DEV) for k in numel]
    B.ws_unpack(plan, ga, ref)
    assert torch.equal(fw, aw) and torch.equal(fm, am), "fused state"
    for a, b in zip(outs, ref):
        assert torch.equal(a, b), "fused weights"

    if not norm_based and R <= 16:
        lists = [[torch.full((k,), 9.0, dtype=odt, device=DEV) for k in numel] for _ in range(R)]
        rw, rm, rv = pw.clone(), pm.clone(), pv.clone()
        gt, wt = B.TensorTable(plan, g), B.TensorTable(plan, lists)
        for r in range(R):
            B.ws_fused_update(plan, r, gt, rw[sl[r]], rm[sl[r]], rv[sl[r]] if has_v else None, hy, wt, None)
        assert torch.equal(rw, aw), "replica kernels: state"
        for k in range(R):
            for a, b in zip(lists[k], ref):
                assert torch.equal(a, b), "replica kernels: weights"
