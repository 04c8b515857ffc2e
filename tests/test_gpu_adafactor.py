"""GPU parity for Adafactor (the optimizer with row / column reduces that the sharding cuts,
Section 4.1): the CUDA library through its C ABI against the CPU oracle's whole-tensor
definition on the same seeded inputs.  Tolerances: 1e-5 under the per-tensor error metric for
the weights (they pass through fp32 row / column sums, as LAMB's pass through fp32 norms),
1e-5 relative for the factored state and the per-tensor scalars, 1e-2 for bf16 outputs."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import ws_oracle as O
from paper_2004_13336_b200 import binding as B
from paper_2004_13336_b200 import workloads as W
from tests._util import TOL_BF16, TOL_LAMB, bf16_to_f64, err, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda"

# matrices with rows longer and shorter than a tile, single rows and columns, 3-D and 4-D tensors,
# vectors (unfactored), tiny and prime sizes, row lengths that are 1/2, 2 and 8 times the 1024 elements
# a CTA covers with one vector per thread
SHAPES = [(1,), (7,), (3, 3, 16, 32), (64, 128), (1031,), (5, 1, 9), (4099, 3), (300, 301), (32,), (20011,),
          (2, 9001), (1, 4500), (4500, 1), (6, 5000), (24, 2048), (3, 8192), (40, 512)]


def _hyper(**kw):
    h = dict(lr=1e-2, beta1=0.0, beta2=0.0, eps=1e-30, weight_decay=0.0, momentum=0.0, grad_scale=1.0, step=10,
             eps2=1e-3, clip_threshold=1.0, decay_exponent=0.8)
    h.update(kw)
    return h


def _setup(shapes, R, gdtype=torch.float32, seed=0, gstd=1e-2, A=32, tile=0, layout="per_tensor", K=None):
    wl = W.Workload("t", list(shapes), R=K or R, opt="adam", hyper={}, grad_dtype=gdtype, grad_std=gstd, seed=seed)
    w, _, _ = W.make_state(wl, DEV)
    g = W.make_grads(wl, DEV)
    plan = B.Plan(shapes, R, A, tile, layout=layout)
    gen = torch.Generator(device="cpu").manual_seed(seed + 99)
    f0 = (torch.rand(plan.factored_elems, generator=gen) * 1e-3 + 1e-6).to(DEV)
    return wl, plan, w, g, f0


def _oracle(shapes, h, w, g, f0):
    hs = O.make_hyper("adafactor", h)
    rows, cols, foff, tot = O.factor_shapes(shapes)
    assert tot == f0.numel()
    f = to_np(f0)
    ow = [to_np(x).reshape(s) for x, s in zip(w, shapes)]
    og = [[to_np(x) for x in gk] for gk in g]
    info = []
    for t in range(len(shapes)):
        vr = f[foff[t]:foff[t] + rows[t]]
        vc = f[foff[t] + rows[t]:foff[t] + rows[t] + cols[t]] if cols[t] else None
        info.append(O.adafactor_tensor(hs, [gk[t] for gk in og], ow[t], vr, vc))
    return ow, f, np.array(info)


def _pack(plan, lists):
    out = []
    for l in lists:
        b = torch.empty(plan.G, dtype=l[0].dtype, device=DEV)
        B.ws_pack(plan, l, b)
        out.append(b)
    return out


def _check(plan, shapes, pw, fs, ws, ow, of, oinfo, tol=TOL_LAMB, d=1.0):
    got = [torch.empty(int(np.prod(s)), dtype=torch.float32, device=DEV) for s in shapes]
    B.ws_unpack(plan, pw, got)
    for t, (a, b) in enumerate(zip(got, ow)):
        e = err(to_np(a), b)
        assert e <= tol, f"w[{t}] {shapes[t]} err {e:.3e}"
    # the factored state per tensor under the same metric: an entry fed by a single element whose R
    # gradient copies cancel carries that fp32 sum's error, far above its own size
    gs = to_np(fs)
    for t, (off, rows, cols) in enumerate(plan.factored_layout()):
        e = err(gs[off:off + rows + cols], of[off:off + rows + cols])
        assert e <= tol, f"state[{t}] {shapes[t]} err {e:.3e}"
    T = plan.T
    coef = ws[:4 * T].view(torch.float32).cpu().numpy().astype(np.float64)
    clip = np.maximum(1.0, oinfo[:, 1] / d)
    np.testing.assert_allclose(coef, oinfo[:, 0] / clip, rtol=1e-5)


@pytest.mark.parametrize("R", [1, 2, 3, 8, 16, 40])
@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
def test_adafactor_matches_oracle_and_fused_equals_unfused(R, gdtype):
    wl, plan, w, g, f0 = _setup(SHAPES, R, gdtype, seed=R + 3)
    h = _hyper()
    ow, of, oinfo = _oracle(SHAPES, h, w, g, f0)
    pw, = _pack(plan, [w])
    pg = _pack(plan, g)
    fs = f0.clone()
    ws = torch.zeros(plan.workspace_bytes("adafactor"), dtype=torch.uint8, device=DEV)
    gath = torch.full((plan.G,), 3.0, dtype=torch.bfloat16, device=DEV)
    B.ws_shard_update(plan, -1, pg, pw, None, fs, B.make_hyper("adafactor", h), gath, ws)
    _check(plan, SHAPES, pw, fs, ws, ow, of, oinfo)
    assert torch.equal(gath, pw.to(torch.bfloat16))
    oplan = O.Plan(wl.numels, R, 32)
    valid = torch.from_numpy(O.pack(oplan, [np.ones(int(n), np.float32) for n in oplan.numel]) != 0).to(DEV)
    assert bool((pw[~valid].view(torch.int32) == 0).all()) and bool((gath[~valid].view(torch.int16) == 0).all())
    # formatting fused in: gradients read from the tensor lists, weights written to the tensors
    fw, = _pack(plan, [w])
    ff = f0.clone()
    outs = [torch.zeros(n, dtype=torch.float32, device=DEV) for n in wl.numels]
    ws2 = torch.full_like(ws, 0xFF)                       # the workspace may hold anything on entry
    B.ws_fused_update(plan, -1, B.TensorTable(plan, g), fw, None, ff, B.make_hyper("adafactor", h),
                      B.TensorTable(plan, [outs]), ws2)
    _check(plan, SHAPES, fw, ff, ws2, ow, of, oinfo)
    got = [torch.empty_like(o) for o in outs]
    B.ws_unpack(plan, fw, got)
    for a, b in zip(outs, got):
        assert torch.equal(a, b)


@pytest.mark.parametrize("tile", [1024, 4096, 16384])
@pytest.mark.parametrize("layout", ["per_tensor", "concat"])
def test_tile_sizes_and_layouts(tile, layout):
    R = 5
    wl, plan, w, g, f0 = _setup(SHAPES, R, seed=21, tile=tile, layout=layout, A=8)
    h = _hyper(step=3, clip_threshold=0.5)
    ow, of, oinfo = _oracle(SHAPES, h, w, g, f0)
    pw, = _pack(plan, [w])
    fs = f0.clone()
    ws = torch.zeros(plan.workspace_bytes("adafactor"), dtype=torch.uint8, device=DEV)
    outs = [torch.zeros(n, dtype=torch.bfloat16, device=DEV) for n in wl.numels]
    B.ws_fused_update(plan, -1, B.TensorTable(plan, g), pw, None, fs, B.make_hyper("adafactor", h),
                      B.TensorTable(plan, [outs]), ws)
    _check(plan, SHAPES, pw, fs, ws, ow, of, oinfo, d=0.5)
    for t, (a, b) in enumerate(zip(outs, ow)):
        assert err(bf16_to_f64(to_np(a)), b) <= TOL_BF16, t


def test_first_step_without_history_and_grad_scale():
    # step 1: beta = 0, the old state is ignored entirely (even NaN-free garbage); mean of 4 copies
    R = 4
    wl, plan, w, g, f0 = _setup(SHAPES, R, seed=5)
    h = _hyper(step=1, grad_scale=0.25, lr=0.5)
    ow, of, oinfo = _oracle(SHAPES, h, w, g, f0)
    pw, = _pack(plan, [w])
    fs = f0.clone()
    ws = torch.zeros(plan.workspace_bytes("adafactor"), dtype=torch.uint8, device=DEV)
    B.ws_shard_update(plan, -1, _pack(plan, g), pw, None, fs, B.make_hyper("adafactor", h), None, ws)
    _check(plan, SHAPES, pw, fs, ws, ow, of, oinfo)


def test_partial_sharding_more_copies_than_shards():
    # 3 groups x 2 shards: 6 gradient copies into a 2-shard plan
    wl, plan, w, g, f0 = _setup(SHAPES, 2, seed=8, K=6)
    h = _hyper()
    ow, of, oinfo = _oracle(SHAPES, h, w, g, f0)
    pw, = _pack(plan, [w])
    fs = f0.clone()
    ws = torch.zeros(plan.workspace_bytes("adafactor"), dtype=torch.uint8, device=DEV)
    B.ws_shard_update(plan, -1, _pack(plan, g), pw, None, fs, B.make_hyper("adafactor", h), None, ws)
    _check(plan, SHAPES, pw, fs, ws, ow, of, oinfo)


def test_three_consecutive_steps_track_the_oracle():
    R = 3
    wl, plan, w, g, f0 = _setup(SHAPES, R, seed=13)
    pw, = _pack(plan, [w])
    fs = f0.clone()
    ws = torch.zeros(plan.workspace_bytes("adafactor"), dtype=torch.uint8, device=DEV)
    ow = [to_np(x) for x in w]
    of = f0.clone()
    for it in range(3):
        wl.seed = 100 + it
        g = W.make_grads(wl, DEV)
        h = _hyper(step=5 + it)
        # oracle continues from its own previous result
        wt = [torch.from_numpy(np.ascontiguousarray(a).ravel()).to(DEV) for a in ow]
        ow, off, oinfo = _oracle(SHAPES, h, wt, g, of)
        of = torch.from_numpy(off).to(DEV)
        B.ws_shard_update(plan, -1, _pack(plan, g), pw, None, fs, B.make_hyper("adafactor", h), None, ws)
    _check(plan, SHAPES, pw, fs, ws, ow, to_np(of), oinfo, tol=3 * TOL_LAMB)


def test_poisoned_pads_and_dirty_workspace_change_nothing():
    R = 7
    wl, plan, w, g, f0 = _setup(SHAPES, R, seed=12)
    oplan = O.Plan(wl.numels, R, 32)
    valid = torch.from_numpy(O.pack(oplan, [np.ones(int(n), np.float32) for n in oplan.numel]) != 0).to(DEV)
    hy = B.make_hyper("adafactor", _hyper())
    h = _hyper()
    ow, of, oinfo = _oracle(SHAPES, h, w, g, f0)
    pw, = _pack(plan, [w])
    pg = _pack(plan, g)
    fs = f0.clone()
    ws = torch.zeros(plan.workspace_bytes("adafactor"), dtype=torch.uint8, device=DEV)
    for b in [pw] + pg:
        b[~valid] = float("nan")
    ws.view(torch.float32)[:] = float("nan")
    B.ws_shard_update(plan, -1, pg, pw, None, fs, hy, None, ws)
    _check(plan, SHAPES, pw, fs, ws, ow, of, oinfo)
    assert bool((pw[~valid].view(torch.int32) == 0).all())


def test_argument_errors():
    R = 2
    wl, plan, w, g, f0 = _setup(SHAPES[:4], R, seed=1)
    pw, = _pack(plan, [w])
    pg = _pack(plan, g)
    ws = torch.zeros(plan.workspace_bytes("adafactor"), dtype=torch.uint8, device=DEV)
    ok = B.make_hyper("adafactor", _hyper())
    for bad, status in ((dict(weight_decay=0.1), 1), (dict(clip_threshold=0.0), 1), (dict(decay_exponent=0.0), 1)):
        with pytest.raises(B.WsError) as e:
            B.ws_shard_update(plan, -1, pg, pw, None, f0, B.make_hyper("adafactor", _hyper(**bad)), None, ws)
        assert e.value.status == status
    with pytest.raises(B.WsError) as e:
        B.ws_shard_update(plan, 0, pg, pw, None, f0, ok, None, ws)             # single shard: refused
    assert e.value.status == 1
    with pytest.raises(B.WsError) as e:
        B.ws_shard_update(plan, -1, pg, pw, None, None, ok, None, ws)          # no factored state
    assert e.value.status == 1
    small = torch.zeros(plan.workspace_bytes("lars"), dtype=torch.uint8, device=DEV)
    with pytest.raises(B.WsError) as e:
        B.ws_shard_update(plan, -1, pg, pw, None, f0, ok, None, small)
    assert e.value.status == 4
    # a workspace that is 16- but not 32-byte aligned: the second pass reads the stored gradient sum with
    # 256-bit loads, so the call is refused on the host and nothing is launched
    big = torch.zeros(plan.workspace_bytes("adafactor") + 64, dtype=torch.uint8, device=DEV)
    shifted = big[16:16 + plan.workspace_bytes("adafactor")]
    assert shifted.data_ptr() % 32 == 16
    w_before = pw.clone()
    with pytest.raises(B.WsError) as e:
        B.ws_shard_update(plan, -1, pg, pw, None, f0, ok, None, shifted)
    assert e.value.status == 2
    torch.cuda.synchronize()
    assert torch.equal(pw, w_before) and float(big.sum()) == 0.0
    lay = plan.factored_layout()
    rows, cols, foff, tot = O.factor_shapes(SHAPES[:4])
    assert [tuple(x) for x in lay] == list(zip(foff.tolist(), rows.tolist(), cols.tolist())) and plan.factored_elems == tot


@pytest.mark.parametrize("case", range(32))
def test_randomised_matrix_shapes_on_both_routes(case):
    """Random lists of 0- to 4-dimensional tensors (row lengths below, at and above what a CTA covers
    with one vector per thread; scalars; empty tensors), shard and copy counts, alignments, tile sizes,
    layouts and dtypes: both routes against the oracle's whole-tensor definition."""
    rng = np.random.default_rng(7000 + case)
    pool = [1, 2, 3, 4, 5, 7, 8, 9, 16, 31, 32, 33, 64, 100, 127, 128, 255, 256, 300, 512, 1000, 1024, 1025, 2048, 4097]

    def shape():
        nd = int(rng.choice([0, 1, 1, 2, 2, 2, 3, 4]))
        s = tuple(int(rng.choice(pool)) for _ in range(nd))
        while int(np.prod(s)) > 400000:
            s = tuple(max(1, d // 2) for d in s)
        if nd and rng.random() < 0.05:
            s = s[:-1] + (0,)
        return s
    shapes = [shape() for _ in range(int(rng.integers(1, 12)))]
    if sum(int(np.prod(s)) for s in shapes) == 0:
        shapes.append((24, 2048))
    R = int(rng.choice([1, 2, 3, 4, 5, 8, 9, 16, 33]))
    K = R if rng.random() < 0.8 else int(rng.choice([1, 2, 6]))
    A, tile = int(rng.choice([8, 16, 32, 64])), int(rng.choice([0, 1024, 2048, 4096]))
    layout = str(rng.choice(["per_tensor", "concat"]))
    gdt = torch.bfloat16 if rng.random() < 0.3 else torch.float32
    odt = torch.bfloat16 if rng.random() < 0.3 else torch.float32
    wl, plan, w, g, f0 = _setup(shapes, R, gdt, seed=case, A=A, tile=tile, layout=layout, K=K)
    h = _hyper(step=int(rng.integers(1, 20)), grad_scale=float(rng.choice([1.0, 0.5])),
               clip_threshold=float(rng.choice([1.0, 0.3])))
    numels = wl.numels
    hs = O.make_hyper("adafactor", h)
    of = to_np(f0)
    ow = [to_np(x) for x in w]
    og = [[to_np(x) for x in gk] for gk in g]
    for t, (off, rows, cols) in enumerate(plan.factored_layout()):
        if numels[t]:
            ref = ow[t].reshape(shapes[t]) if len(shapes[t]) else ow[t]
            O.adafactor_tensor(hs, [gk[t] for gk in og], ref, of[off:off + rows],
                               of[off + rows:off + rows + cols] if cols else None)
            ow[t] = ref.ravel()
    hy = B.make_hyper("adafactor", h)
    for route in ("separate", "fused"):
        pw, = _pack(plan, [w])
        fs = f0.clone()
        ws = torch.full((plan.workspace_bytes("adafactor"),), 0xFF, dtype=torch.uint8, device=DEV)
        outs = [torch.full((n,), 9.0, dtype=odt, device=DEV) for n in numels]
        if route == "separate":
            gath = torch.empty(plan.G, dtype=odt, device=DEV)
            B.ws_shard_update(plan, -1, _pack(plan, g), pw, None, fs, hy, gath, ws)
            B.ws_unpack(plan, gath, outs)
        else:
            B.ws_fused_update(plan, -1, B.TensorTable(plan, g), pw, None, fs, hy, B.TensorTable(plan, [outs]), ws)
        gs = to_np(fs)
        for t, (off, rows, cols) in enumerate(plan.factored_layout()):
            if numels[t] == 0:
                continue
            a = to_np(outs[t])
            a = bf16_to_f64(a) if odt == torch.bfloat16 else a
            # a handful of elements has no tensor-wide scale to be measured against
            tol = TOL_BF16 if odt == torch.bfloat16 else (TOL_LAMB if numels[t] >= 32 else 1e-4)
            assert err(a, ow[t]) <= tol, (route, t, shapes[t])
            assert err(gs[off:off + rows + cols], of[off:off + rows + cols]) <= 10 * TOL_LAMB, (route, t, shapes[t])


@pytest.mark.parametrize("R", [1, 3, 8])
@pytest.mark.parametrize("slice_mode", [0, 1])
def test_stage_by_stage_per_shard_matches_oracle(R, slice_mode):
    """What R replicas would run: the per-shard stages for every shard with the finalize stages in
    between (on one GPU the sums of all shards already meet in the one workspace)."""
    wl, plan, w, g, f0 = _setup(SHAPES, R, seed=R + 31)
    h = _hyper(step=6)
    ow, of, oinfo = _oracle(SHAPES, h, w, g, f0)
    hy = B.make_hyper("adafactor", h)
    pw, = _pack(plan, [w])
    pg = _pack(plan, g)
    fs = f0.clone()
    ws = torch.full((plan.workspace_bytes("adafactor"),), 0xFF, dtype=torch.uint8, device=DEV)
    gath = torch.zeros(plan.G, dtype=torch.bfloat16, device=DEV)
    S = plan.S
    sl = [slice(r * S, (r + 1) * S) for r in range(R)]
    gr = (lambda r: [b[sl[r]] for b in pg]) if slice_mode else (lambda r: pg)
    B.ws_adafactor_stage(plan, B.AF_BEGIN, -1, hy, ws)
    for r in range(R):
        B.ws_adafactor_stage(plan, B.AF_SUMS, r, hy, ws, gbufs=gr(r), w=pw[sl[r]], slice_mode=slice_mode)
    B.ws_adafactor_stage(plan, B.AF_MOMENTS, -1, hy, ws, fstate=fs)
    for r in range(R):
        B.ws_adafactor_stage(plan, B.AF_SUMSQ, r, hy, ws)
    B.ws_adafactor_stage(plan, B.AF_CLIP, -1, hy, ws)
    for r in range(R):
        B.ws_adafactor_stage(plan, B.AF_APPLY, r, hy, ws, w=pw[sl[r]], gathered=gath)
    _check(plan, SHAPES, pw, fs, ws, ow, of, oinfo)
    assert torch.equal(gath, pw.to(torch.bfloat16))
    with pytest.raises(B.WsError) as e:               # a stage number outside the list
        B.ws_adafactor_stage(plan, 9, -1, hy, ws)
    assert e.value.status == 1


def test_step_can_be_captured_in_a_cuda_graph():
    # clear + six kernels of an Adafactor step inside a captured graph: replays track the eager calls
    # (to rounding: the row / column sums are atomic adds)
    R = 3
    wl, plan, w, g, f0 = _setup(SHAPES, R, seed=44)
    hy = B.make_hyper("adafactor", _hyper(step=7))
    pw, = _pack(plan, [w])
    pg = B.PtrList(_pack(plan, g))
    ew, ef, fs = pw.clone(), f0.clone(), f0.clone()
    ws = torch.zeros(plan.workspace_bytes("adafactor"), dtype=torch.uint8, device=DEV)
    for _ in range(2):
        B.ws_shard_update(plan, -1, pg, ew, None, ef, hy, None, ws)
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            B.ws_shard_update(plan, -1, pg, pw, None, fs, hy, None, ws)
    torch.cuda.current_stream().wait_stream(side)
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.allclose(pw, ew, rtol=2e-5, atol=1e-8) and torch.allclose(fs, ef, rtol=2e-4, atol=0)
