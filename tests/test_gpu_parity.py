"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on
the same seeded inputs.  Layout work (pack, unpack, pads, reduce on integers)
is bit-exact; floating-point outputs use the per-tensor error metric of
tests/_util.py with the tolerances 1e-6 (fp32 momentum-SGD / Adam), 1e-5 (LAMB
weights and trust ratios) and 1e-2 (bf16 outputs)."""
import numpy as np
import pytest
import torch

from oracle import ws_oracle as O
from paper_2004_13336_b200 import binding as B
from paper_2004_13336_b200 import workloads as W
from tests._util import TOL_BF16, TOL_FP32, TOL_LAMB, bf16_to_f64, err, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda"

# several tiles (tile = 2048 elements) per piece at small R, ragged tails, tiny and prime sizes
SHAPES = [(1,), (7,), (3, 3, 16, 32), (64, 128), (1031,), (5, 1, 9), (4099, 3), (300, 301), (32,), (20011,)]
RS = [1, 2, 3, 4, 7, 8, 10, 16, 64, 1024]


def _hyper(opt, **kw):
    h = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0, momentum=0.0, grad_scale=1.0, step=10)
    if opt == "sgdm":
        h.update(lr=0.1, momentum=0.9, weight_decay=5e-5)
    if opt == "lamb":
        h.update(eps=1e-6, weight_decay=0.01)
    h.update(kw)
    return h


def _model(shapes, R, gdtype=torch.float32, seed=0, gstd=1e-2):
    wl = W.Workload("t", list(shapes), R=R, opt="adam", hyper={}, grad_dtype=gdtype, grad_std=gstd, seed=seed)
    w, m, v = W.make_state(wl, DEV)
    g = W.make_grads(wl, DEV)
    return wl, w, m, v, g


def _guarded(n, dtype, fill):
    """n-element buffer with 64-element guard zones on both sides."""
    big = torch.full((n + 128,), fill, dtype=dtype, device=DEV)
    return big, big[64:64 + n]


def _guards_intact(big, n, fill):
    ref = torch.full((64,), fill, dtype=big.dtype, device=DEV)
    return bool(torch.equal(big[:64], ref) and torch.equal(big[64 + n:], ref))


def _pack_all(plan, w, m, v, g):
    # the flat buffers start as NaN: ws_pack has to overwrite every element, pads included
    pw = torch.full((plan.G,), float("nan"), dtype=torch.float32, device=DEV)
    pm, pv = pw.clone(), pw.clone()
    B.ws_pack(plan, w, pw)
    B.ws_pack(plan, m, pm)
    B.ws_pack(plan, v, pv)
    pg = []
    for gk in g:
        b = torch.full((plan.G,), float("nan"), dtype=gk[0].dtype, device=DEV)
        B.ws_pack(plan, gk, b)
        pg.append(b)
    assert bool(torch.isfinite(pw).all()) and all(bool(torch.isfinite(b).all()) for b in pg)
    return pw, pm, pv, pg


def _oracle_unsharded(opt, h, w, m, v, g):
    hs = O.make_hyper(opt, h)
    ow, om, ov = [to_np(x) for x in w], [to_np(x) for x in m], [to_np(x) for x in v]
    og = [[to_np(x) for x in gk] for gk in g]
    rho = O.update_unsharded(hs, og, ow, om, ov if opt != "sgdm" else None)
    return ow, om, ov, rho


def _compare_state(oplan, opt, gpu_bufs, ref_lists, tol):
    names = ["w", "m", "v"] if opt != "sgdm" else ["w", "m"]
    for name, buf, ref in zip(names, gpu_bufs, ref_lists):
        got = O.unpack(oplan, to_np(buf))
        for t, (a, b) in enumerate(zip(got, ref)):
            e = err(a, b)
            assert e <= tol, f"{name}[{t}] err {e:.3e} > {tol}"


def _pads_are_zero(oplan, buf):
    valid = O.pack(oplan, [np.ones(int(n), np.float32) for n in oplan.numel]) != 0
    a = to_np(buf)
    bits = a.view(np.uint32) if a.dtype == np.float32 else a
    return bool((bits[~valid] == 0).all())


# ------------------------------------------------------------ pack/unpack ---
@pytest.mark.parametrize("R", RS)
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("A", [8, 32])
def test_pack_unpack_bit_exact(R, dtype, A):
    plan = B.Plan(SHAPES, R, A)
    oplan = O.Plan([int(np.prod(s)) for s in SHAPES], R, A)
    gen = torch.Generator(device=DEV).manual_seed(R)
    tensors = [torch.randn(int(n), device=DEV, generator=gen).to(dtype) for n in oplan.numel]
    fill = 7.0
    big, flat = _guarded(plan.G, dtype, fill)
    B.ws_pack(plan, tensors, flat)
    ref = O.pack(oplan, [to_np(t) for t in tensors])
    assert to_np(flat).tobytes() == ref.tobytes()
    assert _guards_intact(big, plan.G, fill)
    # unpack into guarded, pre-filled tensors
    outs = [_guarded(int(n), dtype, fill) for n in oplan.numel]
    B.ws_unpack(plan, flat, [o[1] for o in outs])
    for (bg, o), t, n in zip(outs, tensors, oplan.numel):
        assert torch.equal(o, t)
        assert _guards_intact(bg, int(n), fill)


def test_unpack_never_reads_pads():
    plan = B.Plan(SHAPES, 7, 32)
    oplan = O.Plan([int(np.prod(s)) for s in SHAPES], 7, 32)
    tensors = [torch.randn(int(n), device=DEV) for n in oplan.numel]
    flat = torch.empty(plan.G, device=DEV)
    B.ws_pack(plan, tensors, flat)
    valid = torch.from_numpy(O.pack(oplan, [np.ones(int(n), np.float32) for n in oplan.numel]) != 0).to(DEV)
    flat[~valid] = float("nan")
    outs = [torch.empty_like(t) for t in tensors]
    B.ws_unpack(plan, flat, outs)
    for o, t in zip(outs, tensors):
        assert torch.equal(o, t)


# ------------------------------------------------------------------ reduce ---
@pytest.mark.parametrize("R", [1, 2, 5, 8, 33, 128])
@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
def test_reduce_is_exact_on_integer_gradients(R, gdtype):
    # plain SGD with lr=1 from w=0: w' = -sum_k g_k, exact for small integers in any order
    plan = B.Plan(SHAPES, R, 8)
    numel = [int(np.prod(s)) for s in SHAPES]
    gen = torch.Generator(device=DEV).manual_seed(R)
    g = [[torch.randint(-64, 64, (n,), device=DEV, generator=gen).to(gdtype) for n in numel] for _ in range(R)]
    w = [torch.zeros(n, device=DEV) for n in numel]
    pw, pm, pv, pg = _pack_all(plan, w, w, w, g)
    h = _hyper("sgdm", lr=1.0, momentum=0.0, weight_decay=0.0)
    B.ws_shard_update(plan, -1, pg, pw, pm, None, B.make_hyper("sgdm", h))
    outs = [torch.empty(n, device=DEV) for n in numel]
    B.ws_unpack(plan, pw, outs)
    for t in range(len(numel)):
        expect = -sum(gk[t].double() for gk in g)
        assert torch.equal(outs[t].double(), expect)


# ------------------------------------------------------------------ update ---
@pytest.mark.parametrize("opt", ["sgdm", "adam", "lamb"])
@pytest.mark.parametrize("R", [1, 2, 3, 4, 8, 10, 16, 64])
@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
def test_update_all_shards_matches_oracle(opt, R, gdtype):
    A = 32
    wl, w, m, v, g = _model(SHAPES, R, gdtype, seed=R)
    plan = B.Plan(SHAPES, R, A)
    oplan = O.Plan(wl.numels, R, A)
    h = _hyper(opt)
    ow, om, ov, orho = _oracle_unsharded(opt, h, w, m, v, g)
    pw, pm, pv, pg = _pack_all(plan, w, m, v, g)
    gath32 = torch.full((plan.G,), 9.0, device=DEV)
    ws = torch.empty(max(16, plan.workspace_bytes(opt)), dtype=torch.uint8, device=DEV)
    B.ws_shard_update(plan, -1, pg, pw, pm, pv if opt != "sgdm" else None, B.make_hyper(opt, h), gath32, ws)
    tol = TOL_LAMB if opt == "lamb" else TOL_FP32
    bufs = [pw, pm, pv] if opt != "sgdm" else [pw, pm]
    refs = [ow, om, ov] if opt != "sgdm" else [ow, om]
    # moments are plain Adam arithmetic for LAMB too
    _compare_state(oplan, opt, bufs[1:], refs[1:], TOL_FP32)
    _compare_state(oplan, opt, bufs[:1], refs[:1], tol)
    for b in bufs:
        assert _pads_are_zero(oplan, b)
    assert torch.equal(gath32, pw)            # fp32 gathered slot == fp32 master, pads +0
    if opt == "lamb":
        rho = B.lamb_ratios(plan, ws).cpu().numpy().astype(np.float64)
        rel = np.abs(rho - np.array(orho)) / np.array(orho)
        assert rel.max() <= TOL_LAMB, rel.max()


@pytest.mark.parametrize("tile", [1024, 4096, 16384])
@pytest.mark.parametrize("opt,gdtype", [("sgdm", torch.float32), ("adam", torch.bfloat16), ("lamb", torch.float32)])
def test_tile_sizes_give_the_same_result(tile, opt, gdtype):
    # pieces of 1, 1.3 and 5.2 tiles at the largest tile size; the result may not depend on the tiling
    shapes = [(3, 7), (40000,), (17, 4099), (9,), (171, 1000)]
    R = 2
    wl, w, m, v, g = _model(shapes, R, gdtype, seed=tile)
    h = B.make_hyper(opt, _hyper(opt))
    outs = []
    for t in (2048, tile):
        plan = B.Plan(shapes, R, 32, t)
        pw, pm, pv, pg = _pack_all(plan, w, m, v, g)
        gath = torch.zeros(plan.G, dtype=torch.bfloat16, device=DEV)
        ws = torch.zeros(max(16, plan.workspace_bytes(opt)), dtype=torch.uint8, device=DEV)
        B.ws_shard_update(plan, -1, pg, pw, pm, pv if opt != "sgdm" else None, h, gath, ws)
        back = [torch.empty_like(x) for x in w]
        B.ws_unpack(plan, pw, back)
        outs.append((pw, pm, pv, gath, back))
    a, b = outs
    assert torch.equal(a[1], b[1]) and torch.equal(a[2], b[2])          # moments: elementwise, tiling-free
    if opt != "lamb":
        assert torch.equal(a[0], b[0]) and torch.equal(a[3], b[3])
    else:   # the norm partial sums are grouped by tile: last-bit differences in rho only
        oplan = O.Plan(wl.numels, R, 32)
        for x, y in zip(O.unpack(oplan, to_np(a[0])), O.unpack(oplan, to_np(b[0]))):
            assert err(x, y) <= 2e-7
    for x, y in zip(a[4], b[4]):
        assert err(to_np(x), to_np(y)) <= 2e-7


@pytest.mark.parametrize("opt", ["sgdm", "adam", "lamb"])
@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
def test_bf16_gathered_copy(opt, gdtype):
    R, A = 4, 32
    wl, w, m, v, g = _model(SHAPES, R, gdtype, seed=11)
    plan = B.Plan(SHAPES, R, A)
    oplan = O.Plan(wl.numels, R, A)
    h = _hyper(opt)
    ow, _, _, _ = _oracle_unsharded(opt, h, w, m, v, g)
    pw, pm, pv, pg = _pack_all(plan, w, m, v, g)
    gath = torch.full((plan.G,), 3.0, dtype=torch.bfloat16, device=DEV)
    ws = torch.empty(max(16, plan.workspace_bytes(opt)), dtype=torch.uint8, device=DEV)
    B.ws_shard_update(plan, -1, pg, pw, pm, pv if opt != "sgdm" else None, B.make_hyper(opt, h), gath, ws)
    # bit-exact self-consistency: bf16 copy == round-to-nearest-even of the fp32 master
    assert torch.equal(gath, pw.to(torch.bfloat16))
    assert to_np(gath).tobytes() == O.f32_to_bf16_bits(to_np(pw)).tobytes()
    assert _pads_are_zero(oplan, gath)
    got = O.unpack(oplan, to_np(gath))
    for a, b in zip(got, ow):
        assert err(bf16_to_f64(a), b) <= TOL_BF16


@pytest.mark.parametrize("opt", ["sgdm", "adam"])
@pytest.mark.parametrize("R", [1, 3, 8])
@pytest.mark.parametrize("slice_mode", [0, 1])
def test_per_shard_calls_equal_all_shard_launch(opt, R, slice_mode):
    wl, w, m, v, g = _model(SHAPES, R, seed=5)
    plan = B.Plan(SHAPES, R, 32)
    h = B.make_hyper(opt, _hyper(opt))
    pw, pm, pv, pg = _pack_all(plan, w, m, v, g)
    aw, am, av = pw.clone(), pm.clone(), pv.clone()
    ga = torch.zeros(plan.G, device=DEV)
    B.ws_shard_update(plan, -1, pg, aw, am, av if opt != "sgdm" else None, h, ga)
    gb = torch.zeros(plan.G, device=DEV)
    S = plan.S
    for r in range(R):
        sl = slice(r * S, (r + 1) * S)
        gr = [b[sl] for b in pg] if slice_mode == 1 else pg
        B.ws_shard_update(plan, r, gr, pw[sl], pm[sl], pv[sl] if opt != "sgdm" else None, h, gb,
                          slice_mode=slice_mode)
    assert torch.equal(aw, pw) and torch.equal(am, pm) and torch.equal(ga, gb)
    if opt == "adam":
        assert torch.equal(av, pv)


@pytest.mark.parametrize("R", [1, 3, 8])
def test_lamb_shard_by_shard_phases(R):
    # (the plan carries no one-launch schedule: the all-shard call runs the same three launches)
    wl, w, m, v, g = _model(SHAPES, R, seed=6)
    plan = B.Plan(SHAPES, R, 32, one_launch=False)
    h = B.make_hyper("lamb", _hyper("lamb"))
    pw, pm, pv, pg = _pack_all(plan, w, m, v, g)
    aw, am, av = pw.clone(), pm.clone(), pv.clone()
    wsa = torch.zeros(plan.workspace_bytes("lamb"), dtype=torch.uint8, device=DEV)
    wsb = torch.zeros_like(wsa)
    ga = torch.zeros(plan.G, dtype=torch.bfloat16, device=DEV)
    gb = torch.zeros_like(ga)
    B.ws_shard_update(plan, -1, pg, aw, am, av, h, ga, wsa)
    S = plan.S
    for r in range(R):
        sl = slice(r * S, (r + 1) * S)
        B.ws_lamb_partial(plan, r, pg, pw[sl], pm[sl], pv[sl], h, wsb)
    B.ws_lamb_finalize(plan, wsb)
    for r in range(R):
        sl = slice(r * S, (r + 1) * S)
        B.ws_lamb_apply(plan, r, pw[sl], pm[sl], pv[sl], h, wsb, gb)
    assert torch.equal(wsa, wsb)
    assert torch.equal(aw, pw) and torch.equal(am, pm) and torch.equal(av, pv) and torch.equal(ga, gb)


@pytest.mark.parametrize("opt", ["sgdm", "adam", "lamb"])
@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
def test_poisoned_pads_never_leak(opt, gdtype):
    R, A = 7, 32
    wl, w, m, v, g = _model(SHAPES, R, gdtype, seed=3)
    plan = B.Plan(SHAPES, R, A)
    oplan = O.Plan(wl.numels, R, A)
    hy = B.make_hyper(opt, _hyper(opt))
    valid = torch.from_numpy(O.pack(oplan, [np.ones(int(n), np.float32) for n in oplan.numel]) != 0).to(DEV)
    results = []
    for poison in (False, True):
        pw, pm, pv, pg = _pack_all(plan, w, m, v, g)
        if poison:
            for b in [pw, pm, pv] + pg:
                b[~valid] = float("nan")
        gath = torch.full((plan.G,), 5.0, dtype=torch.bfloat16, device=DEV)
        ws = torch.zeros(max(16, plan.workspace_bytes(opt)), dtype=torch.uint8, device=DEV)
        B.ws_shard_update(plan, -1, pg, pw, pm, pv if opt != "sgdm" else None, hy, gath, ws)
        out = [pw, pm, gath] + ([pv] if opt != "sgdm" else [])
        if opt == "lamb":
            out.append(B.lamb_ratios(plan, ws).clone())
        results.append(out)
    for a, b in zip(*results):
        assert torch.equal(a, b)
    for b in results[1][:4 if opt != "sgdm" else 3]:
        assert _pads_are_zero(oplan, b)


@pytest.mark.parametrize("R,mode", [(128, "sum"), (1024, "sum"), (1024, "mean")])
def test_many_replicas_small_shards(R, mode):
    # tiny shards (pieces of one alignment unit) and a long gradient sum
    shapes = [(1024,), (1,), (257, 33), (64, 64)]
    wl, w, m, v, g = _model(shapes, R, seed=R, gstd=1e-3)
    plan = B.Plan(shapes, R, 8)
    oplan = O.Plan(wl.numels, R, 8)
    h = _hyper("adam", grad_scale=1.0 if mode == "sum" else 1.0 / R)
    ow, om, ov, _ = _oracle_unsharded("adam", h, w, m, v, g)
    pw, pm, pv, pg = _pack_all(plan, w, m, v, g)
    B.ws_shard_update(plan, -1, pg, pw, pm, pv, B.make_hyper("adam", h))
    _compare_state(oplan, "adam", [pw, pm, pv], [ow, om, ov], TOL_FP32)


def test_argument_errors_are_status_codes():
    import ctypes as C
    plan = B.Plan([(64,), (100,)], 2, 8)
    L = B.lib()
    buf = torch.zeros(plan.G + 8, device=DEV)
    hy = B.make_hyper("adam", _hyper("adam"))
    s = B.ws_state(buf.data_ptr(), buf.data_ptr(), buf.data_ptr())
    ptrs = (C.c_void_p * 2)(buf.data_ptr(), buf.data_ptr())
    g = B.ws_grads(C.cast(ptrs, C.POINTER(C.c_void_p)), 2, 0, 0)
    call = lambda r, gg, ss: L.ws_shard_update(plan.handle, r, C.byref(gg), C.byref(ss), C.byref(hy), None, None, 0, None)
    assert call(2, g, s) == 1 and call(-2, g, s) == 1                       # r out of range
    bad = B.ws_state(buf.data_ptr() + 4, buf.data_ptr(), buf.data_ptr())
    assert call(0, g, bad) == 2                                              # misaligned
    g0 = B.ws_grads(C.cast(ptrs, C.POINTER(C.c_void_p)), 0, 0, 0)
    assert call(0, g0, s) == 1                                               # no gradient copies
    gbig = B.ws_grads(C.cast(ptrs, C.POINTER(C.c_void_p)), 1025, 0, 0)
    assert call(0, gbig, s) in (1, 7)                                        # more copies than the limit
    g1 = B.ws_grads(C.cast(ptrs, C.POINTER(C.c_void_p)), 2, 0, 1)
    assert call(-1, g1, s) == 1                                              # slice mode needs one shard
    gd = B.ws_grads(C.cast(ptrs, C.POINTER(C.c_void_p)), 2, 7, 0)
    assert call(0, gd, s) == 3                                               # dtype
    hl = B.make_hyper("lamb", _hyper("lamb"))
    assert L.ws_shard_update(plan.handle, -1, C.byref(g), C.byref(s), C.byref(hl), None, None, 0, None) == 4
    assert L.ws_shard_update(plan.handle, 0, C.byref(g), C.byref(s), C.byref(hl), None, None, 0, None) == 1
    torch.cuda.synchronize()
    assert float(buf.abs().sum()) == 0.0                                     # nothing was launched


@pytest.mark.parametrize("opt", ["lamb", "lars"])
def test_bad_output_argument_leaves_the_state_untouched(opt):
    # the norm-based optimizers run three launches; a bad `out` (found by the checks of the last one)
    # must be refused before the first launch, or a retry would advance the moments twice
    import ctypes as C
    R = 4
    wl, w, m, v, g = _model(SHAPES[:6], R, seed=9)
    plan = B.Plan(SHAPES[:6], R, 32)
    pw, pm, pv, pg = _pack_all(plan, w, m, v, g)
    before = [pw.clone(), pm.clone(), pv.clone()]
    ws = torch.zeros(plan.workspace_bytes(opt), dtype=torch.uint8, device=DEV)
    h = _lars_hyper() if opt == "lars" else _hyper("lamb")
    hy = B.make_hyper(opt, h)
    gathered = torch.zeros(plan.G + 8, dtype=torch.bfloat16, device=DEV)
    ptrs = (C.c_void_p * R)(*[b.data_ptr() for b in pg])
    gr = B.ws_grads(C.cast(ptrs, C.POINTER(C.c_void_p)), R, 0, 0)
    st = B.ws_state(pw.data_ptr(), pm.data_ptr(), pv.data_ptr() if opt == "lamb" else None)
    for out, status in ((B.ws_out(gathered.data_ptr() + 2, B.WS_BF16), 2), (B.ws_out(gathered.data_ptr(), 9), 3)):
        rc = B.lib().ws_shard_update(plan.handle, -1, C.byref(gr), C.byref(st), C.byref(hy), C.byref(out),
                                     ws.data_ptr(), ws.numel(), None)
        assert rc == status
        if opt == "lamb":
            rc = B.lib().ws_lamb_update_static_scratch(plan.handle, C.byref(gr), C.byref(st), C.byref(hy), C.byref(out), None)
            assert rc == status
    torch.cuda.synchronize()
    assert all(torch.equal(a, b) for a, b in zip((pw, pm, pv), before))
    if opt == "lamb":      # the shard-by-shard LAMB calls refuse another optimizer's hyper-parameters
        ha = B.make_hyper("adam", _hyper("adam"))
        with pytest.raises(B.WsError) as e:
            B.ws_lamb_partial(plan, 0, pg, pw[:plan.S], pm[:plan.S], pv[:plan.S], ha, ws)
        assert e.value.status == 1
        with pytest.raises(B.WsError) as e:
            B.ws_lamb_apply(plan, 0, pw[:plan.S], pm[:plan.S], pv[:plan.S], ha, ws)
        assert e.value.status == 1


@pytest.mark.parametrize("opt", ["sgdm", "adam", "lamb"])
@pytest.mark.parametrize("fused", [False, True])
def test_checkpoint_round_trip_equals_uninterrupted_run(opt, fused):
    # Section 4.2: the auxiliary variables stay sharded between steps and are gathered only when a
    # checkpoint needs them (the "unsharding program"); restoring shards them again (the "sharding
    # program").  Step, unpack w / m / v to checkpoint-shaped tensors, pack them into fresh buffers of a
    # fresh plan, step again: bit for bit the state of two uninterrupted steps.
    R = 5
    wl, w, m, v, g = _model(SHAPES, R, seed=44)
    g2 = W.make_grads(W.Workload("t", list(SHAPES), R=R, opt="adam", hyper={}, grad_std=1e-2, seed=45), DEV)
    has_v = opt != "sgdm"

    def step(plan, bufs, grads, stepno):
        hy = B.make_hyper(opt, _hyper(opt, step=stepno))
        ws = torch.zeros(max(32, plan.workspace_bytes(opt)), dtype=torch.uint8, device=DEV)
        pw, pm, pv = bufs
        if fused:
            outs = [torch.zeros_like(x) for x in w]
            B.ws_fused_update(plan, -1, B.TensorTable(plan, grads), pw, pm, pv if has_v else None, hy,
                              B.TensorTable(plan, [outs]), ws)
        else:
            pg = []
            for gk in grads:
                b = torch.empty(plan.G, device=DEV)
                B.ws_pack(plan, gk, b)
                pg.append(b)
            B.ws_shard_update(plan, -1, pg, pw, pm, pv if has_v else None, hy, None, ws)

    plan = B.Plan(SHAPES, R, 32)
    a = list(_pack_all(plan, w, m, v, [])[:3])
    step(plan, a, g, 10)
    step(plan, a, g2, 11)                                   # uninterrupted
    b = list(_pack_all(plan, w, m, v, [])[:3])
    step(plan, b, g, 10)
    ckpt = [[torch.empty_like(x) for x in w] for _ in range(3)]
    for buf, lst in zip(b, ckpt):
        B.ws_unpack(plan, buf, lst)                         # the checkpoint: tensors in their own shapes
    del plan
    plan2 = B.Plan(SHAPES, R, 32)                           # a restarted job plans again
    c = list(_pack_all(plan2, ckpt[0], ckpt[1], ckpt[2], [])[:3])
    step(plan2, c, g2, 11)
    torch.cuda.synchronize()
    for x, y in zip(a[:3 if has_v else 2], c):
        assert torch.equal(x, y)


# ------------------------------------------------- fused formatting path ---
def _views_with_guards(numels, dtype, fill, misalign):
    """One buffer per tensor with 64-element guards; `misalign` shifts the view by 16 bytes so
    that tensors are 16- but not 32-byte aligned."""
    shift = (16 // torch.empty(0, dtype=dtype).element_size()) if misalign else 0
    bigs, views = [], []
    for n in numels:
        big = torch.full((n + 128 + shift,), fill, dtype=dtype, device=DEV)
        bigs.append(big)
        views.append(big[64 + shift:64 + shift + n])
    return bigs, views


@pytest.mark.parametrize("opt", ["sgdm", "adam", "lamb"])
@pytest.mark.parametrize("R", [1, 3, 8, 40])
@pytest.mark.parametrize("gdtype,odtype,misalign", [(torch.float32, torch.float32, False),
                                                     (torch.bfloat16, torch.bfloat16, False),
                                                     (torch.float32, torch.bfloat16, True),
                                                     (torch.bfloat16, torch.float32, True)])
def test_fused_update_equals_pack_update_unpack(opt, R, gdtype, odtype, misalign):
    wl, w, m, v, g = _model(SHAPES, R, gdtype, seed=R + 50)
    plan = B.Plan(SHAPES, R, 32)
    h = B.make_hyper(opt, _hyper(opt))
    numels = wl.numels
    # reference: pack every gradient list, update, unpack the gathered buffer
    pw, pm, pv, pg = _pack_all(plan, w, m, v, g)
    fw, fm, fv = pw.clone(), pm.clone(), pv.clone()
    gathered = torch.zeros(plan.G, dtype=odtype, device=DEV)
    ws = torch.zeros(max(16, plan.workspace_bytes(opt)), dtype=torch.uint8, device=DEV)
    B.ws_shard_update(plan, -1, pg, pw, pm, pv if opt != "sgdm" else None, h, gathered, ws)
    ref_w = [torch.empty(n, dtype=odtype, device=DEV) for n in numels]
    B.ws_unpack(plan, gathered, ref_w)
    # fused: gradient tensors (optionally only 16-byte aligned) in, weight tensors out
    gb = [_views_with_guards(numels, gdtype, float("nan"), misalign) for _ in range(R)]
    for (bigs, views), gk in zip(gb, g):
        for dst, src in zip(views, gk):
            dst.copy_(src)
    wb_bigs, wb_views = _views_with_guards(numels, odtype, 7.0, misalign)
    gt = B.TensorTable(plan, [views for _, views in gb])
    wt = B.TensorTable(plan, [wb_views])
    assert gt.c.min_align >= (32 if not misalign else 16)
    ws2 = torch.zeros_like(ws)
    B.ws_fused_update(plan, -1, gt, fw, fm, fv if opt != "sgdm" else None, h, wt, ws2)
    # With 16-byte-only alignment the fused kernel runs its 128-bit variant while the packed path
    # runs the 256-bit one: elementwise results are identical, but LAMB's norm partial sums are
    # grouped differently, so rho (hence w') may differ in the last bit.
    exact = not (opt == "lamb" and misalign)
    assert torch.equal(fm, pm)
    if opt != "sgdm":
        assert torch.equal(fv, pv)
    if exact:
        assert torch.equal(fw, pw)
    else:
        assert err(to_np(fw), to_np(pw)) <= 2e-7
    shift = (16 // ref_w[0].element_size()) if misalign else 0
    for big, view, ref, n in zip(wb_bigs, wb_views, ref_w, numels):
        if exact:
            assert torch.equal(view, ref)
        else:
            assert err(to_np(view.float()), to_np(ref.float())) <= (TOL_BF16 if odtype == torch.bfloat16 else 2e-7)
        guard = torch.full((64 + shift,), 7.0, dtype=odtype, device=DEV)
        assert torch.equal(big[:64 + shift], guard) and torch.equal(big[64 + shift + n:], guard[:64])


@pytest.mark.parametrize("opt", ["sgdm", "adam"])
def test_fused_update_shard_by_shard(opt):
    R = 5
    wl, w, m, v, g = _model(SHAPES, R, seed=77)
    plan = B.Plan(SHAPES, R, 32)
    h = B.make_hyper(opt, _hyper(opt))
    pw, pm, pv, _ = _pack_all(plan, w, m, v, g)
    aw, am, av = pw.clone(), pm.clone(), pv.clone()
    gt = B.TensorTable(plan, g)
    out_all = [torch.zeros_like(x) for x in w]
    out_one = [torch.zeros_like(x) for x in w]
    B.ws_fused_update(plan, -1, gt, aw, am, av if opt != "sgdm" else None, h, B.TensorTable(plan, [out_all]))
    wt = B.TensorTable(plan, [out_one])
    S = plan.S
    for r in range(R):
        sl = slice(r * S, (r + 1) * S)
        B.ws_fused_update(plan, r, gt, pw[sl], pm[sl], pv[sl] if opt != "sgdm" else None, h, wt)
    assert torch.equal(aw, pw) and torch.equal(am, pm)
    for a, b in zip(out_all, out_one):
        assert torch.equal(a, b)


def test_fused_update_matches_oracle_unsharded():
    # the fused path straight against the plain definition (no packed buffers anywhere)
    wl = W.scaled_down(W.resnet50(), 48)
    w, m, v = W.make_state(wl, DEV)
    g = W.make_grads(wl, DEV)
    plan = B.Plan(wl.shapes, wl.R, 32)
    ow, om, _, _ = _oracle_unsharded(wl.opt, wl.hyper, w, m, v, g)
    pw, pm, pv, _ = _pack_all(plan, w, m, v, [])
    outs = [torch.zeros_like(x) for x in w]
    B.ws_fused_update(plan, -1, B.TensorTable(plan, g), pw, pm, None, B.make_hyper(wl.opt, wl.hyper),
                      B.TensorTable(plan, [outs]))
    for a, b in zip(outs, ow):
        assert err(to_np(a), b) <= TOL_FP32


@pytest.mark.parametrize("opt", ["sgdm", "adam", "lamb"])
def test_empty_tensors_in_the_list(opt):
    shapes = [(64, 33), (0,), (5, 0, 2), (4099,), (0, 7)]
    R = 3
    wl, w, m, v, g = _model(shapes, R, seed=9)
    plan = B.Plan(shapes, R, 32)
    oplan = O.Plan(wl.numels, R, 32)
    assert plan.S == oplan.S
    h = _hyper(opt)
    ow, om, ov, orho = _oracle_unsharded(opt, h, w, m, v, g)
    pw, pm, pv, pg = _pack_all(plan, w, m, v, g)
    fw, fm, fv = pw.clone(), pm.clone(), pv.clone()
    ws = torch.zeros(max(16, plan.workspace_bytes(opt)), dtype=torch.uint8, device=DEV)
    B.ws_shard_update(plan, -1, pg, pw, pm, pv if opt != "sgdm" else None, B.make_hyper(opt, h), None, ws)
    tol = TOL_LAMB if opt == "lamb" else TOL_FP32
    _compare_state(oplan, opt, [pw, pm, pv][:3 if opt != "sgdm" else 2], [ow, om, ov][:3 if opt != "sgdm" else 2], tol)
    if opt == "lamb":
        rho = B.lamb_ratios(plan, ws).cpu().numpy()
        assert rho[1] == 1.0 and rho[2] == 1.0 and rho[4] == 1.0
    outs = [torch.full_like(x, 3.0) for x in w]
    B.ws_fused_update(plan, -1, B.TensorTable(plan, g), fw, fm, fv if opt != "sgdm" else None,
                      B.make_hyper(opt, h), B.TensorTable(plan, [outs]), ws)
    assert torch.equal(fw, pw) and torch.equal(fm, pm)
    back = [torch.empty_like(x) for x in w]
    B.ws_unpack(plan, pw, back)
    for a, b in zip(outs, back):
        assert torch.equal(a, b)


@pytest.mark.parametrize("opt", ["sgdm", "adam", "lamb", "lars"])
def test_empty_tensors_in_the_concatenated_layout(opt):
    # empty tensors first, in the middle and last; 4 x 32-element alignment units in total, so with
    # R = 4 the concatenation fills the shards exactly and the trailing empty tensor owns no tile at all
    shapes = [(0,), (32,), (5, 0, 2), (64,), (0, 7), (32,), (100, 0)]
    R = 4
    wl, w, m, v, g = _model(shapes, R, seed=19)
    plan = B.Plan(shapes, R, 32, layout="concat")
    oplan = O.FlatPlan(wl.numels, R, 32)
    assert plan.S == oplan.S == 32
    h = _lars_hyper() if opt == "lars" else _hyper(opt)
    has_v = opt in ("adam", "lamb")
    ow, om, ov, _ = _oracle_unsharded(opt, h, w, m, v, g)
    nan = float("nan")
    pw, pm, pv = (torch.full((plan.G,), nan, device=DEV) for _ in range(3))
    for src, dst in ((w, pw), (m, pm), (v, pv)):
        B.ws_pack(plan, src, dst)                       # must overwrite every element of the flat buffer
    assert bool(torch.isfinite(pw).all())
    pg = []
    for gk in g:
        b = torch.full((plan.G,), nan, device=DEV)
        B.ws_pack(plan, gk, b)
        pg.append(b)
    fw, fm, fv = pw.clone(), pm.clone(), pv.clone()
    ws = torch.full((max(16, plan.workspace_bytes(opt)),), 0xFF, dtype=torch.uint8, device=DEV)
    B.ws_shard_update(plan, -1, pg, pw, pm, pv if has_v else None, B.make_hyper(opt, h), None, ws)
    tol = TOL_LAMB if opt in ("lamb", "lars") else TOL_FP32
    for t, (a, b) in enumerate(zip(O.unpack_flat(oplan, to_np(pw)), ow)):
        assert err(a, b) <= tol, t
    outs = [torch.full_like(x, 3.0) for x in w]
    B.ws_fused_update(plan, -1, B.TensorTable(plan, g), fw, fm, fv if has_v else None, B.make_hyper(opt, h),
                      B.TensorTable(plan, [outs]), torch.full_like(ws, 0xFF))
    assert torch.equal(fw, pw) and torch.equal(fm, pm)
    back = [torch.empty_like(x) for x in w]
    B.ws_unpack(plan, pw, back)
    for a, b in zip(outs, back):
        assert torch.equal(a, b)


def test_step_can_be_captured_in_a_cuda_graph():
    # calls take pointers and a stream, allocate nothing and never synchronise, so a whole step
    # (here: the fused update, and pack + update + unpack) can be captured once and replayed
    wl, w, m, v, g = _model(SHAPES, 4, seed=4)
    plan = B.Plan(SHAPES, 4, 32)
    hy = B.make_hyper("adam", _hyper("adam"))
    pw, pm, pv, pg = _pack_all(plan, w, m, v, g)
    ew, em, ev = pw.clone(), pm.clone(), pv.clone()
    outs = [torch.zeros_like(x) for x in w]
    gt, wt = B.TensorTable(plan, g), B.TensorTable(plan, [outs])
    gl = B.PtrList(pg)
    B.ws_fused_update(plan, -1, gt, ew, em, ev, hy, wt)        # eager reference: two steps
    B.ws_fused_update(plan, -1, gt, ew, em, ev, hy, wt)
    expect = [o.clone() for o in outs]
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for gk, b in zip(g, pg):
                B.ws_pack(plan, gk, b)
            B.ws_shard_update(plan, -1, gl, pw, pm, pv, hy)
            B.ws_unpack(plan, pw, outs)
    torch.cuda.current_stream().wait_stream(side)
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(pw, ew) and torch.equal(pm, em) and torch.equal(pv, ev)
    for a, b in zip(outs, expect):
        assert torch.equal(a, b)


@pytest.mark.parametrize("opt,R", [("lamb", 3), ("lamb", 8), ("lars", 3)])
def test_multi_launch_steps_can_be_captured_in_a_cuda_graph(opt, R):
    # the norm-based optimizers are three launches joined by programmatic dependent launch - or, for LAMB
    # with 8 copies, a clear of the counters and the one kernel: the captured graph replays to the same
    # bits as the eager calls (fixed-order sums)
    wl, w, m, v, g = _model(SHAPES, R, seed=14, gstd=1e-3)
    plan = B.Plan(SHAPES, R, 32)
    h = _lars_hyper() if opt == "lars" else _hyper(opt)
    hy = B.make_hyper(opt, h)
    pw, pm, pv, pg = _pack_all(plan, w, m, v, g)
    ew, em, ev = pw.clone(), pm.clone(), pv.clone()
    gl = B.PtrList(pg)
    ws = torch.zeros(plan.workspace_bytes(opt), dtype=torch.uint8, device=DEV)
    sv, esv = (pv, ev) if opt == "lamb" else (None, None)
    for _ in range(2):                                           # eager reference: two steps
        B.ws_shard_update(plan, -1, gl, ew, em, esv, hy, None, ws)
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            B.ws_shard_update(plan, -1, gl, pw, pm, sv, hy, None, ws)
    torch.cuda.current_stream().wait_stream(side)
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(pw, ew) and torch.equal(pm, em)
    if opt == "lamb" and R == 8:
        off = plan.sync_status_offset()
        assert int(ws[off:off + 4].view(torch.int32).item()) == 0


@pytest.mark.parametrize("opt", ["sgdm", "adam", "lamb"])
@pytest.mark.parametrize("groups,M", [(2, 4), (5, 2), (3, 1)])
def test_partial_sharding_more_gradient_copies_than_shards(opt, groups, M):
    # Section 5.2: groups of replicas shard M ways each; shard j sums all groups*M copies
    K = groups * M
    wl, w, m, v, g = _model(SHAPES, K, seed=K)
    plan = B.Plan(SHAPES, M, 32)
    oplan = O.Plan(wl.numels, M, 32)
    h = _hyper(opt)
    ow, om, ov, _ = _oracle_unsharded(opt, h, w, m, v, g)          # plain definition over all K copies
    pw, pm, pv, pg = _pack_all(plan, w, m, v, g)
    assert len(pg) == K and plan.R == M
    fw, fm, fv = pw.clone(), pm.clone(), pv.clone()
    ws = torch.zeros(max(16, plan.workspace_bytes(opt)), dtype=torch.uint8, device=DEV)
    B.ws_shard_update(plan, -1, pg, pw, pm, pv if opt != "sgdm" else None, B.make_hyper(opt, h), None, ws)
    n = 3 if opt != "sgdm" else 2
    _compare_state(oplan, opt, [pw, pm, pv][:n], [ow, om, ov][:n], TOL_LAMB if opt == "lamb" else TOL_FP32)
    outs = [torch.zeros_like(x) for x in w]
    B.ws_fused_update(plan, -1, B.TensorTable(plan, g), fw, fm, fv if opt != "sgdm" else None,
                      B.make_hyper(opt, h), B.TensorTable(plan, [outs]), ws)
    assert torch.equal(fw, pw) and torch.equal(fm, pm)


# ------------------------------------------------------------------- LARS ---
def _lars_hyper(**kw):
    return _hyper("sgdm", lr=10.0, momentum=0.9, weight_decay=5e-5, trust_coeff=0.001, **kw)


@pytest.mark.parametrize("R", [1, 2, 3, 8, 16, 40])
@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
def test_lars_matches_oracle_and_fused_equals_unfused(R, gdtype):
    wl, w, m, v, g = _model(SHAPES, R, gdtype, seed=R + 7, gstd=1e-3)
    plan = B.Plan(SHAPES, R, 32)
    oplan = O.Plan(wl.numels, R, 32)
    h = _lars_hyper()
    ow, om, _, orate = _oracle_unsharded("lars", h, w, m, v, g)
    pw, pm, _, pg = _pack_all(plan, w, m, v, g)
    fw, fm = pw.clone(), pm.clone()
    ws = torch.zeros(plan.workspace_bytes("lars"), dtype=torch.uint8, device=DEV)
    gath = torch.full((plan.G,), 3.0, dtype=torch.bfloat16, device=DEV)
    B.ws_shard_update(plan, -1, pg, pw, pm, None, B.make_hyper("lars", h), gath, ws)
    # the local rate carries fp32 norm error (~1e-7), so w' and m' get the LAMB-class tolerance
    _compare_state(oplan, "sgdm", [pw, pm], [ow, om], TOL_LAMB)
    rate = B.lamb_ratios(plan, ws).cpu().numpy().astype(np.float64)
    rel = np.abs(rate - np.array(orate)) / np.array(orate)
    assert rel.max() <= TOL_LAMB, rel.max()
    assert _pads_are_zero(oplan, pw) and _pads_are_zero(oplan, pm) and _pads_are_zero(oplan, gath)
    assert torch.equal(gath, pw.to(torch.bfloat16))
    outs = [torch.zeros(n, dtype=torch.bfloat16, device=DEV) for n in wl.numels]
    ws2 = torch.zeros_like(ws)
    B.ws_fused_update(plan, -1, B.TensorTable(plan, g), fw, fm, None, B.make_hyper("lars", h),
                      B.TensorTable(plan, [outs]), ws2)
    assert torch.equal(fw, pw) and torch.equal(fm, pm)
    ref = [torch.zeros_like(o) for o in outs]
    B.ws_unpack(plan, gath, ref)
    for a, b in zip(outs, ref):
        assert torch.equal(a, b)


@pytest.mark.parametrize("opt", ["lamb", "lars"])
@pytest.mark.parametrize("R", [1, 2, 3, 8, 16, 32, 40])
@pytest.mark.parametrize("gdtype,layout,fused", [(torch.float32, "per_tensor", False), (torch.bfloat16, "per_tensor", True),
                                                 (torch.float32, "concat", True), (torch.bfloat16, "concat", False)])
def test_one_launch_update_equals_three_launches(opt, R, gdtype, layout, fused):
    # The all-shard LAMB / LARS update as ONE kernel (plan with its one-launch schedule) against
    # the three launches (phase 1, combination, phase 2): same elementwise arithmetic, the norm sums grouped
    # by work item instead of by tile, so ratios agree to rounding; the status word stays 0; two steps in
    # a row (the second finds the first's counters and flags in the workspace).  The one-kernel route is
    # taken for LAMB with 8 to 32 gradient copies; every other case runs the three launches on both plans.
    shapes = SHAPES + [(1024, 512), (0,), (70001,)]
    wl, w, m, v, g = _model(shapes, R, gdtype, seed=R + 31, gstd=1e-3 if opt == "lars" else 1e-2)
    p1 = B.Plan(shapes, R, 32, layout=layout)
    p3 = B.Plan(shapes, R, 32, layout=layout, one_launch=False)
    assert p1.sched_buf is not None and p3.sched_buf is None
    h = _lars_hyper() if opt == "lars" else _hyper("lamb")
    has_v = opt == "lamb"
    bufs = {}
    for name, plan in (("one", p1), ("three", p3)):
        pw, pm, pv, pg = _pack_all(plan, w, m, v, g)
        ws = torch.full((max(32, plan.workspace_bytes(opt)),), 0xA5, dtype=torch.uint8, device=DEV)   # dirty workspace
        outs = [torch.zeros(n, dtype=torch.bfloat16, device=DEV) for n in wl.numels]
        gathered = torch.zeros(plan.G, dtype=torch.bfloat16, device=DEV)
        gt = B.TensorTable(plan, g) if fused else None
        wt = B.TensorTable(plan, [outs]) if fused else None
        for step in (10, 11):
            hy = B.make_hyper(opt, dict(h, step=step))
            if fused:
                B.ws_fused_update(plan, -1, gt, pw, pm, pv if has_v else None, hy, wt, ws)
            else:
                B.ws_shard_update(plan, -1, pg, pw, pm, pv if has_v else None, hy, gathered, ws)
        torch.cuda.synchronize()
        if not fused:
            B.ws_unpack(plan, gathered, outs)
        bufs[name] = (pw, pm, pv, outs, B.lamb_ratios(plan, ws).clone(), ws)
    if opt == "lamb" and 8 <= R <= 32:         # (otherwise both plans run the three launches)
        off = p1.sync_status_offset()
        assert int(bufs["one"][5][off:off + 4].view(torch.int32).item()) == 0
    a, b = bufs["one"], bufs["three"]
    tol = 3e-7
    assert err(to_np(a[0]), to_np(b[0])) <= tol and err(to_np(a[1]), to_np(b[1])) <= tol
    if has_v:
        assert torch.equal(a[2], b[2])
    ra, rb = a[4].cpu().numpy().astype(np.float64), b[4].cpu().numpy().astype(np.float64)
    assert np.all(np.abs(ra / rb - 1.0) <= 1e-6)
    for x, y in zip(a[3], b[3]):
        assert err(to_np(x.float()), to_np(y.float())) <= TOL_BF16
    assert _pads_are_zero(O.Plan(wl.numels, R, 32), a[0]) if layout == "per_tensor" else True


@pytest.mark.parametrize("R", [1, 3, 8])
def test_lars_shard_by_shard_phases(R):
    # what R replicas would run (phase 1 per shard, finalize, phase 2 per shard) equals the all-shard call
    wl, w, m, v, g = _model(SHAPES, R, seed=16, gstd=1e-3)
    plan = B.Plan(SHAPES, R, 32, one_launch=False)
    h = B.make_hyper("lars", _lars_hyper())
    pw, pm, _, pg = _pack_all(plan, w, m, v, g)
    aw, am = pw.clone(), pm.clone()
    wsa = torch.zeros(plan.workspace_bytes("lars"), dtype=torch.uint8, device=DEV)
    wsb = torch.zeros_like(wsa)
    ga = torch.zeros(plan.G, dtype=torch.bfloat16, device=DEV)
    gb = torch.zeros_like(ga)
    B.ws_shard_update(plan, -1, pg, aw, am, None, h, ga, wsa)
    S = plan.S
    for r in range(R):
        sl = slice(r * S, (r + 1) * S)
        B.ws_lars_partial(plan, r, pg, pw[sl], pm[sl], h, wsb)
    B.ws_lars_finalize(plan, h, wsb)
    for r in range(R):
        sl = slice(r * S, (r + 1) * S)
        B.ws_lars_apply(plan, r, pw[sl], pm[sl], h, wsb, gb)
    assert torch.equal(wsa, wsb)
    assert torch.equal(aw, pw) and torch.equal(am, pm) and torch.equal(ga, gb)
    with pytest.raises(B.WsError) as e:           # the LARS calls refuse another optimizer's hyper-parameters
        B.ws_lars_finalize(plan, B.make_hyper("lamb", _hyper("lamb")), wsb)
    assert e.value.status == 1


def test_lars_poisoned_pads_and_error_codes():
    import ctypes as C
    R = 5
    wl, w, m, v, g = _model(SHAPES, R, seed=12, gstd=1e-3)
    plan = B.Plan(SHAPES, R, 32)
    oplan = O.Plan(wl.numels, R, 32)
    hy = B.make_hyper("lars", _lars_hyper())
    valid = torch.from_numpy(O.pack(oplan, [np.ones(int(n), np.float32) for n in oplan.numel]) != 0).to(DEV)
    res = []
    for poison in (False, True):
        pw, pm, _, pg = _pack_all(plan, w, m, v, g)
        ws = torch.zeros(plan.workspace_bytes("lars"), dtype=torch.uint8, device=DEV)
        if poison:
            for b in [pw, pm] + pg:
                b[~valid] = float("nan")
            ws.view(torch.float32)[:] = float("nan")       # the workspace may hold anything on entry
        B.ws_shard_update(plan, -1, pg, pw, pm, None, hy, None, ws)
        res.append((pw, pm, B.lamb_ratios(plan, ws).clone()))
    for a, b in zip(*res):
        assert torch.equal(a, b)
    # too small a workspace and a single-shard call are refused before any launch
    pw, pm, _, pg = _pack_all(plan, w, m, v, g)
    small = torch.zeros(plan.workspace_bytes("lamb"), dtype=torch.uint8, device=DEV)
    with pytest.raises(B.WsError) as e:
        B.ws_shard_update(plan, -1, pg, pw, pm, None, hy, None, small)
    assert e.value.status == 4
    with pytest.raises(B.WsError) as e:
        B.ws_shard_update(plan, 0, pg, pw, pm, None, hy, None, torch.zeros(plan.workspace_bytes("lars"), dtype=torch.uint8, device=DEV))
    assert e.value.status == 1


# ------------------------------------------------------- host-buffer step ---
@pytest.mark.parametrize("opt,gdtype,odtype", [("sgdm", torch.float32, torch.float32),
                                               ("adam", torch.bfloat16, torch.bfloat16),
                                               ("lamb", torch.float32, torch.bfloat16)])
def test_step_host_from_pinned_arenas_matches_oracle(opt, gdtype, odtype):
    R = 3
    wl, w, m, v, g = _model(SHAPES, R, gdtype, seed=31)
    plan = B.Plan(SHAPES, R, 32)
    h = _hyper(opt)
    ow, _, _, _ = _oracle_unsharded(opt, h, w, m, v, g)
    pw, pm, pv, _ = _pack_all(plan, w, m, v, [])
    n_el, numels = plan.arena_elems, wl.numels
    host_g = []
    for gk in g:                                   # one pinned arena per replica, tensors back to back
        a = torch.zeros(n_el, dtype=gdtype).pin_memory()
        for dst, src in zip(plan.arena_views(a, numels), gk):
            dst.copy_(src)
        host_g.append(a)
    host_w = torch.full((n_el,), 5.0, dtype=odtype).pin_memory()
    stage = torch.empty(n_el, dtype=gdtype, device=DEV)
    packed = [torch.empty(plan.G, dtype=gdtype, device=DEV) for _ in range(R)]
    dev_w = torch.empty(n_el, dtype=odtype, device=DEV)
    gathered = torch.empty(plan.G, dtype=odtype, device=DEV) if odtype != torch.float32 else None
    ws = torch.zeros(max(16, plan.workspace_bytes(opt)), dtype=torch.uint8, device=DEV)
    B.ws_step_host(plan, host_g, stage, packed, pw, pm, pv if opt != "sgdm" else None, B.make_hyper(opt, h),
                   dev_w, host_w, gathered, ws)
    torch.cuda.synchronize()
    tol = TOL_BF16 if odtype == torch.bfloat16 else (TOL_LAMB if opt == "lamb" else TOL_FP32)
    for got, ref in zip(plan.arena_views(host_w, numels), ow):
        got = to_np(got)
        assert err(bf16_to_f64(got) if odtype == torch.bfloat16 else got, ref) <= tol


@pytest.mark.parametrize("opt,gdtype,odtype", [("sgdm", torch.float32, torch.float32),
                                               ("adam", torch.bfloat16, torch.bfloat16),
                                               ("lamb", torch.float32, torch.float32)])
def test_fused_update_on_pinned_host_tensors_matches_oracle(opt, gdtype, odtype):
    # the end-to-end step without staging copies: the gradient and weight tensors are pinned host memory,
    # the kernel reads and writes them over PCIe; the sharded state stays on the device
    R = 8 if opt == "lamb" else 3
    wl, w, m, v, g = _model(SHAPES, R, gdtype, seed=37)
    plan = B.Plan(SHAPES, R, 32)
    h = _hyper(opt)
    ow, om, _, _ = _oracle_unsharded(opt, h, w, m, v, g)
    pw, pm, pv, _ = _pack_all(plan, w, m, v, [])
    n_el, numels = plan.arena_elems, wl.numels
    host_g = []
    for gk in g:
        a = torch.zeros(n_el, dtype=gdtype).pin_memory()
        for dst, src in zip(plan.arena_views(a, numels), gk):
            dst.copy_(src)
        host_g.append(a)
    host_w = torch.zeros(n_el, dtype=odtype).pin_memory()
    master = odtype == torch.float32
    if master:                                     # fp32 weights: the host tensors are the master copy
        for dst, src in zip(plan.arena_views(host_w, numels), w):
            dst.copy_(src)
    gt = B.TensorTable(plan, [plan.arena_views(a, numels) for a in host_g], device=DEV)
    wt = B.TensorTable(plan, [plan.arena_views(host_w, numels)], device=DEV)
    ws = torch.zeros(max(32, plan.workspace_bytes(opt)), dtype=torch.uint8, device=DEV)
    B.ws_fused_update(plan, -1, gt, None if master else pw, pm, pv if opt != "sgdm" else None,
                      B.make_hyper(opt, h), wt, ws)
    torch.cuda.synchronize()
    tol = TOL_BF16 if odtype == torch.bfloat16 else (TOL_LAMB if opt == "lamb" else TOL_FP32)
    for got, ref in zip(plan.arena_views(host_w, numels), ow):
        got = to_np(got)
        assert err(bf16_to_f64(got) if odtype == torch.bfloat16 else got, ref) <= tol


def test_more_than_1024_tensors():
    # tensor pointers travel in kernel parameters in chunks of 1024: a list longer than that
    # takes several pack launches; the update and the fused route see one table
    rng = np.random.default_rng(0)
    shapes = [(int(n),) for n in rng.integers(1, 300, 1100)] + [(5000,), (3, 7)]
    R = 3
    wl, w, m, v, g = _model(shapes, R, seed=2)
    plan = B.Plan(shapes, R, 8)
    oplan = O.Plan(wl.numels, R, 8)
    flat = torch.empty(plan.G, device=DEV)
    B.ws_pack(plan, w, flat)
    assert to_np(flat).tobytes() == O.pack(oplan, [to_np(x) for x in w]).tobytes()
    back = [torch.zeros_like(x) for x in w]
    B.ws_unpack(plan, flat, back)
    for a, b in zip(back, w):
        assert torch.equal(a, b)
    h = _hyper("adam")
    ow, om, ov, _ = _oracle_unsharded("adam", h, w, m, v, g)
    pw, pm, pv, pg = _pack_all(plan, w, m, v, g)
    fw, fm, fv = pw.clone(), pm.clone(), pv.clone()
    B.ws_shard_update(plan, -1, pg, pw, pm, pv, B.make_hyper("adam", h))
    _compare_state(oplan, "adam", [pw, pm, pv], [ow, om, ov], TOL_FP32)
    outs = [torch.zeros_like(x) for x in w]
    B.ws_fused_update(plan, -1, B.TensorTable(plan, g), fw, fm, fv, B.make_hyper("adam", h), B.TensorTable(plan, [outs]))
    assert torch.equal(fw, pw)
    B.ws_unpack(plan, pw, back)
    for a, b in zip(outs, back):
        assert torch.equal(a, b)


# ------------------------------------------- concatenated layout (Section 5.2) ---
CONCAT_SHAPES = SHAPES + [(0,), (77,)]


@pytest.mark.parametrize("R", [1, 2, 3, 7, 16, 64, 1024])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_concat_pack_unpack_bit_exact(R, dtype):
    numel = [int(np.prod(s)) for s in CONCAT_SHAPES]
    plan = B.Plan(CONCAT_SHAPES, R, 32, layout="concat")
    oplan = O.FlatPlan(numel, R, 32)
    assert (plan.S, plan.G) == (oplan.S, oplan.G)
    gen = torch.Generator(device=DEV).manual_seed(R)
    tensors = [torch.randn(n, device=DEV, generator=gen).to(dtype) for n in numel]
    big, flat = _guarded(plan.G, dtype, 7.0)
    B.ws_pack(plan, tensors, flat)
    assert to_np(flat).tobytes() == O.pack_flat(oplan, [to_np(t) for t in tensors]).tobytes()
    assert _guards_intact(big, plan.G, 7.0)
    outs = [_guarded(n, dtype, 7.0) for n in numel]
    B.ws_unpack(plan, flat, [o[1] for o in outs])
    for (bg, o), t, n in zip(outs, tensors, numel):
        assert torch.equal(o, t) and _guards_intact(bg, n, 7.0)


@pytest.mark.parametrize("opt", ["sgdm", "adam", "lamb", "lars"])
@pytest.mark.parametrize("R", [1, 3, 8, 40])
@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
def test_concat_update_matches_oracle_on_both_routes(opt, R, gdtype):
    wl, w, m, v, g = _model(CONCAT_SHAPES, R, gdtype, seed=R + 3, gstd=1e-3)
    plan = B.Plan(CONCAT_SHAPES, R, 32, layout="concat")
    oplan = O.FlatPlan(wl.numels, R, 32)
    h = _lars_hyper() if opt == "lars" else _hyper(opt)
    has_v = opt in ("adam", "lamb")
    ow, om, ov, orho = _oracle_unsharded(opt, h, w, m, v, g)
    pw, pm, pv, pg = _pack_all(plan, w, m, v, g)
    valid = torch.from_numpy(oplan.tensor_map() >= 0).to(DEV)
    for b in [pw, pm, pv] + pg:                      # pads may hold anything on entry
        b[~valid] = float("nan")
    fw, fm, fv = pw.clone(), pm.clone(), pv.clone()
    ws = torch.zeros(max(16, plan.workspace_bytes(opt)), dtype=torch.uint8, device=DEV)
    gath = torch.full((plan.G,), 3.0, dtype=torch.bfloat16, device=DEV)
    B.ws_shard_update(plan, -1, pg, pw, pm, pv if has_v else None, B.make_hyper(opt, h), gath, ws)
    tol = TOL_LAMB if opt in ("lamb", "lars") else TOL_FP32
    for name, buf, ref in (("w", pw, ow), ("m", pm, om), ("v", pv, ov)):
        if name == "v" and not has_v:
            continue
        for t, (a, b) in enumerate(zip(O.unpack_flat(oplan, to_np(buf)), ref)):
            assert err(a, b) <= (TOL_FP32 if name == "v" else tol), f"{name}[{t}]"
        assert (to_np(buf).view(np.uint32)[~valid.cpu().numpy()] == 0).all()
    assert torch.equal(gath, pw.to(torch.bfloat16))
    if opt in ("lamb", "lars"):
        rho = B.lamb_ratios(plan, ws).cpu().numpy().astype(np.float64)
        assert (np.abs(rho - np.array(orho)) / np.array(orho)).max() <= TOL_LAMB
    # formatting fused in: same state bit for bit, weights equal to the unpacked gathered buffer
    outs = [torch.zeros(n, dtype=torch.bfloat16, device=DEV) for n in wl.numels]
    ws2 = torch.zeros_like(ws)
    B.ws_fused_update(plan, -1, B.TensorTable(plan, g), fw, fm, fv if has_v else None, B.make_hyper(opt, h),
                      B.TensorTable(plan, [outs]), ws2)
    assert torch.equal(fw, pw) and torch.equal(fm, pm)
    ref = [torch.zeros_like(o) for o in outs]
    B.ws_unpack(plan, gath, ref)
    for a, b in zip(outs, ref):
        assert torch.equal(a, b)


@pytest.mark.parametrize("slice_mode", [0, 1])
def test_concat_shard_by_shard_equals_all_shards(slice_mode):
    R = 6
    wl, w, m, v, g = _model(CONCAT_SHAPES, R, seed=8)
    plan = B.Plan(CONCAT_SHAPES, R, 32, layout="concat")
    h = B.make_hyper("adam", _hyper("adam"))
    pw, pm, pv, pg = _pack_all(plan, w, m, v, g)
    aw, am, av = pw.clone(), pm.clone(), pv.clone()
    ga, gb = torch.zeros(plan.G, device=DEV), torch.zeros(plan.G, device=DEV)
    B.ws_shard_update(plan, -1, pg, aw, am, av, h, ga)
    S = plan.S
    for r in range(R):
        sl = slice(r * S, (r + 1) * S)
        gr = [b[sl] for b in pg] if slice_mode == 1 else pg
        B.ws_shard_update(plan, r, gr, pw[sl], pm[sl], pv[sl], h, gb, slice_mode=slice_mode)
    assert torch.equal(aw, pw) and torch.equal(am, pm) and torch.equal(av, pv) and torch.equal(ga, gb)


def test_tiny_workload_against_stored_oracle_values():
    # config "tiny": CPU-drawn inputs, GPU update (both routes), compared with the values the oracle
    # wrote to tests/golden/tiny_adam_expected.txt
    import os
    wl = W.tiny()
    w, m, v = W.make_state(wl, "cpu")
    g = W.make_grads(wl, "cpu")
    w, m, v = ([x.to(DEV) for x in lst] for lst in (w, m, v))
    g = [[x.to(DEV) for x in gk] for gk in g]
    plan = B.Plan(wl.shapes, wl.R, 32)
    pw, pm, pv, pg = _pack_all(plan, w, m, v, g)
    fw, fm, fv = pw.clone(), pm.clone(), pv.clone()
    hy = B.make_hyper(wl.opt, wl.hyper)
    B.ws_shard_update(plan, -1, pg, pw, pm, pv, hy)
    outs = [torch.zeros_like(x) for x in w]
    B.ws_fused_update(plan, -1, B.TensorTable(plan, g), fw, fm, fv, hy, B.TensorTable(plan, [outs]))
    assert torch.equal(fw, pw) and torch.equal(fm, pm) and torch.equal(fv, pv)
    rows = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "tiny_adam_expected.txt")) as f:
        for line in f:
            if not line.startswith("#"):
                p = line.split()
                rows[(p[0], int(p[1]))] = (int(p[2]), float(p[3]), float(p[4]), [float.fromhex(h) for h in p[5:9]])
    for name, buf in (("w", pw), ("m", pm), ("v", pv)):
        got = [torch.zeros_like(x) for x in w]
        B.ws_unpack(plan, buf, got)
        for t, x in enumerate(got):
            x = to_np(x).astype(np.float64)
            n, s, s2, picks = rows[(name, t)]
            rms = np.sqrt(s2 / n)
            assert x.size == n
            assert abs(np.sum(x * x) - s2) <= 4e-6 * s2
            for i, ref in zip((0, n // 3, 2 * n // 3, n - 1), picks):
                assert abs(x[i] - ref) <= TOL_FP32 * max(abs(ref), rms), (name, t, i)


@pytest.mark.parametrize("case", range(24))
def test_randomised_configurations_on_both_routes(case):
    """Random tensor lists, shard and copy counts, alignments, tile sizes, dtypes, optimizers and
    layouts: the separate-kernel route against the oracle's plain definition, the fused route
    bit-equal to the separate-kernel route."""
    rng = np.random.default_rng(1000 + case)
    T = int(rng.integers(1, 14))
    numel = [int(x) for x in rng.choice([0, 1, 5, 8, 33, 250, 1023, 2048, 4100, 9001, 30011], T)]
    if sum(numel) == 0:
        numel[0] = 17
    shapes = [(n,) for n in numel]
    M = int(rng.choice([1, 2, 3, 4, 7, 8, 12, 40]))
    K = M * int(rng.choice([1, 1, 2]))                     # sometimes more copies than shards
    A = int(rng.choice([8, 32, 128]))
    tile = int(rng.choice([0, 1024, 2048]))
    opt = str(rng.choice(["sgdm", "adam", "lamb", "lars"]))
    gdtype = torch.bfloat16 if rng.integers(2) else torch.float32
    odtype = torch.bfloat16 if rng.integers(2) else torch.float32
    layout = "concat" if rng.integers(2) else "per_tensor"
    wl, w, m, v, g = _model(shapes, K, gdtype, seed=case, gstd=1e-3)
    plan = B.Plan(shapes, M, A, tile, layout=layout)
    h = _lars_hyper() if opt == "lars" else _hyper(opt)
    has_v = opt in ("adam", "lamb")
    ow, om, ov, _ = _oracle_unsharded(opt, h, w, m, v, g)
    pw, pm, pv, pg = _pack_all(plan, w, m, v, g)
    fw, fm, fv = pw.clone(), pm.clone(), pv.clone()
    ws = torch.zeros(max(16, plan.workspace_bytes(opt)), dtype=torch.uint8, device=DEV)
    gath = torch.zeros(plan.G, dtype=odtype, device=DEV)
    B.ws_shard_update(plan, -1, pg, pw, pm, pv if has_v else None, B.make_hyper(opt, h), gath, ws)
    tol = TOL_LAMB if opt in ("lamb", "lars") else TOL_FP32
    for name, buf, ref in (("w", pw, ow), ("m", pm, om), ("v", pv, ov)):
        if name == "v" and not has_v:
            continue
        got = [torch.zeros_like(x) for x in w]
        B.ws_unpack(plan, buf, got)
        for t, (a, b) in enumerate(zip(got, ref)):
            assert err(to_np(a), b) <= (TOL_FP32 if name == "v" else tol), (name, t)
    outs = [torch.full((n,), 9.0, dtype=odtype, device=DEV) for n in numel]
    ws2 = torch.zeros_like(ws)
    B.ws_fused_update(plan, -1, B.TensorTable(plan, g), fw, fm, fv if has_v else None, B.make_hyper(opt, h),
                      B.TensorTable(plan, [outs]), ws2)
    assert torch.equal(fw, pw) and torch.equal(fm, pm) and (not has_v or torch.equal(fv, pv))
    ref = [torch.zeros_like(o) for o in outs]
    B.ws_unpack(plan, gath, ref)
    for a, b in zip(outs, ref):
        assert torch.equal(a, b)


@pytest.mark.parametrize("layout", ["per_tensor", "concat"])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_pack_sets_equals_pack_per_set(layout, dtype):
    R = 5
    wl, w, m, v, g = _model(SHAPES, R, dtype, seed=13)
    plan = B.Plan(SHAPES, R, 32, layout=layout)
    one = []
    for gk in g:
        b = torch.empty(plan.G, dtype=dtype, device=DEV)
        B.ws_pack(plan, gk, b)
        one.append(b)
    many = [torch.full((plan.G,), 3.0, dtype=dtype, device=DEV) for _ in range(R)]
    B.ws_pack_sets(plan, B.TensorTable(plan, g), many)
    for a, b in zip(one, many):
        assert torch.equal(a, b)


@pytest.mark.parametrize("opt", ["lamb", "lars"])
def test_zero_norm_tensors_get_ratio_one(opt):
    # the degenerate cases of the norm-based optimizers: an all-zero weight tensor and a tensor
    # whose update direction (LAMB) or gradient (LARS) is all zero
    shapes = [(300, 7), (5000,), (64,), (2100,)]
    R = 3
    wl, w, m, v, g = _model(shapes, R, seed=21, gstd=1e-3)
    w[1].zero_()                                   # zero weight norm
    for gk in g:
        gk[3].zero_()                              # zero gradient ...
    m[3].zero_()
    v[3].zero_()                                   # ... and zero moments
    h = _lars_hyper() if opt == "lars" else _hyper("lamb", weight_decay=0.0)
    plan = B.Plan(shapes, R, 32)
    oplan = O.Plan(wl.numels, R, 32)
    ow, om, ov, orho = _oracle_unsharded(opt, h, w, m, v, g)
    assert orho[1] == 1.0 and orho[3] == 1.0
    pw, pm, pv, pg = _pack_all(plan, w, m, v, g)
    ws = torch.zeros(plan.workspace_bytes(opt), dtype=torch.uint8, device=DEV)
    B.ws_shard_update(plan, -1, pg, pw, pm, pv if opt == "lamb" else None, B.make_hyper(opt, h), None, ws)
    rho = B.lamb_ratios(plan, ws).cpu().numpy()
    assert rho[1] == 1.0 and rho[3] == 1.0
    _compare_state(oplan, "sgdm", [pw, pm], [ow, om], TOL_LAMB)
    if opt == "lamb":                              # (LARS still applies its weight decay at rate 1)
        got = O.unpack(oplan, to_np(pw))
        assert (got[3] == to_np(w[3])).all()       # nothing to apply: weights unchanged bit for bit


# ------------------------- one kernel per replica over every replica's tensors ---
@pytest.mark.parametrize("opt,gdtype,odtype", [("sgdm", torch.float32, torch.float32),
                                               ("adam", torch.bfloat16, torch.bfloat16),
                                               ("adam", torch.float32, torch.float32)])
@pytest.mark.parametrize("R", [2, 5, 8])
def test_replica_kernels_over_all_replicas_tensors(opt, gdtype, odtype, R):
    """What R replicas with peer-mapped tensors would run, emulated on one GPU by R independent
    launches: replica r's single kernel reads its slice of all R gradient lists (the reduce-scatter),
    updates shard r, and writes the new weights into all R replicas' weight lists (the all-gather).
    Afterwards every replica's weight tensors hold the unsharded result."""
    wl, w, m, v, g = _model(SHAPES, R, gdtype, seed=40 + R)
    plan = B.Plan(SHAPES, R, 32)
    oplan = O.Plan(wl.numels, R, 32)
    h = _hyper(opt)
    ow, om, ov, _ = _oracle_unsharded(opt, h, w, m, v, g)
    pw, pm, pv, _ = _pack_all(plan, w, m, v, [])
    fill = -7.0
    bigs, lists = [], []
    for k in range(R):                 # replica k's weight tensors, with guard zones
        bl = [_guarded(n, odtype, fill) for n in wl.numels]
        bigs.append([b for b, _ in bl])
        lists.append([vw for _, vw in bl])
    gtab = B.TensorTable(plan, g)
    wtab = B.TensorTable(plan, lists)
    hy = B.make_hyper(opt, h)
    S = plan.S
    for r in range(R):                 # independent launches: none waits for another
        sl = slice(r * S, (r + 1) * S)
        B.ws_fused_update(plan, r, gtab, pw[sl], pm[sl], pv[sl] if opt == "adam" else None, hy, wtab, None)
    _compare_state(oplan, opt, [pw, pm, pv], [ow, om, ov], TOL_FP32)
    ref = [torch.empty(n, dtype=odtype, device=DEV) for n in wl.numels]
    B.ws_unpack(plan, pw.to(odtype) if odtype != torch.float32 else pw, ref)
    for k in range(R):
        for t, (a, b) in enumerate(zip(lists[k], ref)):
            assert torch.equal(a, b), (k, t)
            assert _guards_intact(bigs[k][t], wl.numels[t], fill), (k, t)
    # more weight lists than gradient sets, or several lists under a two-phase optimizer: refused
    with pytest.raises(B.WsError) as e:
        B.ws_fused_update(plan, 0, B.TensorTable(plan, g[:1]), pw[:S], pm[:S], pv[:S], hy, wtab, None)
    assert e.value.status == 1
