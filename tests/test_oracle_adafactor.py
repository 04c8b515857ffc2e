"""Pins for the oracle's Adafactor (the paper's example of an optimizer whose reduce operators
collapse a sharded dimension, Section 4.1): torch.optim.Adafactor in float64, closed forms,
invariants of the formula, and the sharded route against the unsharded one."""
import numpy as np
import pytest
import torch

from oracle import ws_oracle as O


def _hyper(**kw):
    h = dict(lr=1e-2, beta1=0.0, beta2=0.0, eps=1e-30, weight_decay=0.0, momentum=0.0, grad_scale=1.0,
             step=10, eps2=1e-3, clip_threshold=1.0, decay_exponent=0.8)
    h.update(kw)
    return O.make_hyper("adafactor", h), h


def _state(rng, shape):
    if len(shape) >= 2:
        rows, cols = int(np.prod(shape[:-1])), shape[-1]
        return (np.abs(rng.normal(0, 1e-4, rows)).astype(np.float32) * cols,
                np.abs(rng.normal(0, 1e-4, cols)).astype(np.float32) * rows)
    return np.abs(rng.normal(0, 1e-6, shape[0])).astype(np.float32), None


@pytest.mark.parametrize("shape", [(7, 5), (1, 9), (33, 1), (64, 48), (301,), (1,)])
@pytest.mark.parametrize("K", [1, 4])
def test_matches_torch_optim_adafactor_float64(shape, K):
    """Three consecutive steps against the library.  The library keeps row and column MEANS and
    clamps instead of adding eps1; with eps1 = 0 here and a clamp far below every value there,
    both are the same function (the means' factors cancel in Rv Cv^T / sum(Rv))."""
    rng = np.random.default_rng(len(shape) * 100 + shape[0] + K)
    w = rng.normal(0, 0.05, shape).astype(np.float32)
    vr, vc = _state(rng, shape)
    p = torch.nn.Parameter(torch.tensor(w.astype(np.float64)))
    opt = torch.optim.Adafactor([p], lr=1e-2, beta2_decay=-0.8, eps=(1e-200, 1e-3), d=1.0, weight_decay=0.0,
                                foreach=False)
    t0 = 4
    st = opt.state[p]
    st["step"] = torch.tensor(float(t0))
    if len(shape) >= 2:
        st["row_var"] = torch.tensor(vr.astype(np.float64) / shape[-1]).reshape(shape[0], 1)
        st["col_var"] = torch.tensor(vc.astype(np.float64) / shape[0]).reshape(1, shape[1])
        st["variance"] = None
    else:
        st["row_var"] = st["col_var"] = None
        st["variance"] = torch.tensor(vr.astype(np.float64))
    for it in range(3):
        g = [rng.normal(0, 1e-2, shape).astype(np.float32) for _ in range(K)]
        p.grad = torch.tensor(sum(x.astype(np.float64) for x in g))
        opt.step()
        hs, _ = _hyper(step=t0 + 1 + it, eps=0.0)
        O.adafactor_tensor(hs, g, w, vr, vc)
        # the oracle stores fp32 after every step, the library carries float64: a few fp32 ulps
        np.testing.assert_allclose(w, p.detach().numpy(), rtol=1e-6, atol=1e-9)
        if len(shape) >= 2:
            np.testing.assert_allclose(vr / shape[-1], st["row_var"].numpy().ravel(), rtol=1e-6)
            np.testing.assert_allclose(vc / shape[0], st["col_var"].numpy().ravel(), rtol=1e-6)
        else:
            np.testing.assert_allclose(vr, st["variance"].numpy(), rtol=1e-6)


def test_rank_one_squared_gradient_gives_sign_update():
    # G^2 = a b^T exactly and t = 1 (beta = 0, no history): V = G^2, U = sign(G), RMS(U) = 1, no
    # clipping; the step is alpha sign(G) with alpha = max(eps2, RMS(w)) min(lr, 1)
    rng = np.random.default_rng(3)
    a = 2.0 ** rng.integers(-6, 3, 12)
    b = 2.0 ** rng.integers(-6, 3, 20)
    sgn = rng.choice([-1.0, 1.0], (12, 20))
    g = (sgn * np.outer(a, b)).astype(np.float32)
    w0 = rng.normal(0, 0.5, (12, 20)).astype(np.float32)
    for lr, eps2 in ((1e-2, 1e-3), (3.0, 1e-3), (1e-2, 10.0)):
        hs, _ = _hyper(step=1, eps=0.0, lr=lr, eps2=eps2)
        w, vr, vc = w0.copy(), np.full(12, 7.0, np.float32), np.full(20, 9.0, np.float32)
        alpha, rms_u, sum_r = O.adafactor_tensor(hs, [g], w, vr, vc)
        rms_w = np.sqrt(np.mean(w0.astype(np.float64) ** 2))
        assert abs(alpha - max(eps2, rms_w) * min(lr, 1.0)) < 1e-15
        assert abs(rms_u - 1.0) < 1e-12
        np.testing.assert_allclose(w, w0 - alpha * sgn, rtol=2e-7, atol=1e-9)
        np.testing.assert_allclose(vr, (np.outer(a, b) ** 2).sum(1), rtol=1e-7)     # history forgotten at t = 1
        np.testing.assert_allclose(vc, (np.outer(a, b) ** 2).sum(0), rtol=1e-7)
        assert abs(sum_r - (np.outer(a, b) ** 2).sum()) / sum_r < 1e-12


def test_decay_step_size_and_eps1_closed_forms():
    # zero gradient: the sums are eps1 per element, U = 0, weights stay
    hs, _ = _hyper(step=8, eps=1e-30)
    w0 = np.linspace(-1, 1, 24, dtype=np.float32).reshape(4, 6)
    w, vr, vc = w0.copy(), np.full(4, 0.5, np.float32), np.full(6, 0.25, np.float32)
    O.adafactor_tensor(hs, [np.zeros((4, 6), np.float32)], w, vr, vc)
    beta = 1.0 - 8.0 ** -0.8
    np.testing.assert_array_equal(w, w0)
    np.testing.assert_allclose(vr, beta * 0.5 + (1 - beta) * 6e-30, rtol=1e-7)
    np.testing.assert_allclose(vc, beta * 0.25 + (1 - beta) * 4e-30, rtol=1e-7)
    # vector, constant inputs: v' = beta v + (1-beta) g^2, u = g / sqrt(v'), RMS(u) = |u| clipped to d
    n, g0, v0, c = 50, 0.02, 1e-4, 0.3
    for d in (1.0, 0.25, 100.0):
        hs, _ = _hyper(step=100, eps=0.0, clip_threshold=d, lr=0.05)
        w, v = np.full(n, c, np.float32), np.full(n, v0, np.float32)
        alpha, rms_u, _ = O.adafactor_tensor(hs, [np.full(n, g0, np.float32)], w, v, None)
        beta = 1.0 - 100.0 ** -0.8
        vn = beta * np.float32(v0) + (1 - beta) * float(np.float32(g0)) ** 2
        u = float(np.float32(g0)) / np.sqrt(vn)
        assert abs(rms_u - u) / u < 1e-12
        assert abs(alpha - float(np.float32(c)) * 0.05) < 1e-12         # min(lr, 1/sqrt(100)) = 0.05
        np.testing.assert_allclose(v, vn, rtol=1e-7)
        np.testing.assert_allclose(w, float(np.float32(c)) - alpha * u / max(1.0, u / d), rtol=2e-7)


def test_invariants_scale_free_first_step_and_clipped_step_length():
    rng = np.random.default_rng(11)
    shape = (17, 23)
    w0 = rng.normal(0, 0.1, shape).astype(np.float32)
    g = rng.normal(0, 1e-2, shape).astype(np.float32)
    outs = []
    for scale in (1.0, 256.0):
        hs, h = _hyper(step=1, eps=0.0)
        w, vr, vc = w0.copy(), np.zeros(17, np.float32), np.zeros(23, np.float32)
        alpha, rms_u, _ = O.adafactor_tensor(hs, [(g * scale).astype(np.float32)], w, vr, vc)
        outs.append(w)
        # the applied step has RMS alpha * min(RMS(U), d): never longer than alpha * d
        step_rms = np.sqrt(np.mean((w.astype(np.float64) - w0) ** 2))
        assert abs(step_rms - alpha * min(rms_u, 1.0)) / step_rms < 1e-4
    np.testing.assert_allclose(outs[0], outs[1], rtol=1e-6)
    # summed gradient copies and grad_scale: K copies at scale 1/K equal one copy
    hs1, _ = _hyper()
    hs4, _ = _hyper(grad_scale=0.25)
    wa, wb = w0.copy(), w0.copy()
    sa, sb = [np.ones(17, np.float32), np.ones(23, np.float32)], [np.ones(17, np.float32), np.ones(23, np.float32)]
    O.adafactor_tensor(hs1, [g], wa, *sa)
    O.adafactor_tensor(hs4, [g, g, g, g], wb, *sb)
    np.testing.assert_array_equal(wa, wb)
    np.testing.assert_array_equal(sa[0], sb[0])


def test_row_and_column_sums_are_not_swapped():
    # a gradient with one hot row: only that row's Rv moves, every Cv moves by the same amount
    g = np.zeros((5, 3), np.float32)
    g[2] = [1.0, 2.0, 3.0]
    hs, _ = _hyper(step=1, eps=0.0)
    w, vr, vc = np.ones((5, 3), np.float32), np.zeros(5, np.float32), np.zeros(3, np.float32)
    O.adafactor_tensor(hs, [g], w, vr, vc)
    np.testing.assert_array_equal(vr, [0, 0, 14.0, 0, 0])
    np.testing.assert_array_equal(vc, [1.0, 4.0, 9.0])
    # a 3-D tensor is the matrix of its last dimension against the leading ones together
    rng = np.random.default_rng(2)
    g3 = rng.normal(0, 1, (2, 4, 6)).astype(np.float32)
    w3a, w3b = np.ones((2, 4, 6), np.float32), np.ones((8, 6), np.float32)
    ra, ca, rb, cb = (np.zeros(8, np.float32), np.zeros(6, np.float32), np.zeros(8, np.float32), np.zeros(6, np.float32))
    O.adafactor_tensor(hs, [g3], w3a, ra, ca)
    O.adafactor_tensor(hs, [g3.reshape(8, 6)], w3b, rb, cb)
    np.testing.assert_array_equal(w3a.reshape(8, 6), w3b)
    np.testing.assert_array_equal(ra, rb)


SHAPES = [(1,), (9,), (8, 8), (5, 1, 9), (37, 13), (3, 3, 16, 32), (2050,), (1, 77), (64, 3)]


def _run_both(R, A, K, bf16, seed, poison=False, out_dtype=None, **hk):
    rng = np.random.default_rng(seed)
    numel = [int(np.prod(s)) for s in SHAPES]
    plan = O.Plan(numel, R, A)
    hs, _ = _hyper(**hk)
    w = [rng.normal(0, 0.05, n).astype(np.float32) for n in numel]
    g = [[rng.normal(0, 1e-2, n).astype(np.float32) for n in numel] for _ in range(K)]
    if bf16:
        g = [[O.f32_to_bf16_bits(x) for x in gk] for gk in g]
    rows, cols, foff, tot = O.factor_shapes(SHAPES)
    f0 = np.abs(rng.normal(0, 1e-3, tot)).astype(np.float32)
    # unsharded: tensor by tensor
    uw = [x.copy().reshape(s) for x, s in zip(w, SHAPES)]
    fu = f0.copy()
    infos = []
    for t, s in enumerate(SHAPES):
        vr = fu[foff[t]:foff[t] + rows[t]]
        vc = fu[foff[t] + rows[t]:foff[t] + rows[t] + cols[t]] if cols[t] else None
        infos.append(O.adafactor_tensor(hs, [gk[t] for gk in g], uw[t], vr, vc))
    # sharded
    pw = O.pack(plan, w)
    gp = [O.pack(plan, gk) for gk in g]
    if poison:
        valid = O.pack(plan, [np.ones(n, np.float32) for n in numel]) > 0
        pw[~valid] = np.float32(1e30)
        for b in gp:
            b[~valid] = 0x7F80 if bf16 else np.float32(np.inf)
    fs = f0.copy()
    gathered, info = O.adafactor_sharded(hs, plan, SHAPES, gp, pw, fs, out_dtype)
    return plan, (uw, fu, np.array(infos)), (pw, fs, gathered, info)


@pytest.mark.parametrize("R", [1, 3, 8, 64])
@pytest.mark.parametrize("bf16", [False, True])
def test_sharded_equals_unsharded(R, bf16):
    # the sharded route cuts rows and columns across shards and combines per-shard partial sums:
    # same result as whole tensors up to the order of the double-precision sums
    plan, (uw, fu, iu), (pw, fs, gathered, info) = _run_both(R, 8, 3, bf16, seed=R, out_dtype=O.BF16)
    np.testing.assert_allclose(info, iu, rtol=1e-12)
    np.testing.assert_allclose(fs, fu, rtol=2e-7)
    for a, b in zip(uw, O.unpack(plan, pw)):
        a = a.ravel()
        assert (np.abs(a.astype(np.float64) - b) <= np.spacing(np.abs(a))).all()
    np.testing.assert_array_equal(gathered, O.f32_to_bf16_bits(pw))


def test_poisoned_pads_never_leak():
    # pads holding inf / 1e30 in the gradients and weights: masked by location, results unchanged
    _, _, clean = _run_both(7, 32, 2, False, seed=1, out_dtype=O.F32)
    _, _, dirty = _run_both(7, 32, 2, False, seed=1, out_dtype=O.F32, poison=True)
    for a, b in zip(clean, dirty):
        assert a.tobytes() == b.tobytes()


@pytest.mark.parametrize("R", [1, 3, 8])
def test_one_replicas_stages_compose_to_the_sharded_update(R):
    """Section 4.1, reduces that collapse a dimension the sharding cuts: every replica reduces what its
    shard holds and the replicas combine their results.  The per-replica stage functions, run for
    r = 0..R-1 with the row / column sums and the scalar sums added over r in ascending order, must give
    bit for bit what the all-shard routine gives (one gradient copy: the reduce-scatter has summed them)."""
    shapes = [(7,), (5, 9), (64, 33), (3, 3, 4, 8), (1031,), (1, 40), (40, 1)]
    numel = [int(np.prod(s)) for s in shapes]
    rng = np.random.default_rng(70 + R)
    h = dict(lr=1e-2, beta1=0.0, beta2=0.0, eps=1e-30, weight_decay=0.0, momentum=0.0, grad_scale=0.5, step=7,
             eps2=1e-3, clip_threshold=1.0, decay_exponent=0.8)
    hs = O.make_hyper("adafactor", h)
    w = [rng.normal(0, 0.02, n).astype(np.float32) for n in numel]
    g = [rng.normal(0, 1e-2, n).astype(np.float32) for n in numel]
    p = O.Plan(numel, R, 8)
    rows, cols, foff, F = O.factor_shapes(shapes)
    f0 = rng.uniform(1e-6, 1e-3, F).astype(np.float32)
    pw, pg = O.pack(p, w), O.pack(p, g)
    aw, af = pw.copy(), f0.copy()
    gathered, info = O.adafactor_sharded(hs, p, shapes, [pg], aw, af, O.BF16)
    S = p.S
    reps = [O.AdafactorReplica(hs, p, shapes, r) for r in range(R)]
    for r, rep in enumerate(reps):
        rep.sums(pg[r * S:(r + 1) * S], pw[r * S:(r + 1) * S])
    acc, sw = np.zeros(F), np.zeros(p.T)
    for rep in reps:                           # ascending r
        acc += rep.acc
        sw += rep.pw
    fs = f0.copy()
    for rep in reps:                           # the small factored state is replicated
        fr = f0.copy()
        rep.moments(acc, fr)
        fs = fr
        rep.sumsq()
    su = np.zeros(p.T)
    for rep in reps:
        su += rep.pu
    slots = []
    for r, rep in enumerate(reps):
        alpha, clip = rep.step_sizes(sw, su)
        slots.append(rep.apply(alpha, clip, pw[r * S:(r + 1) * S], O.BF16))
    assert fs.tobytes() == af.tobytes()
    assert pw.tobytes() == aw.tobytes()
    assert np.concatenate(slots).tobytes() == gathered.tobytes()
    assert alpha.tobytes() == np.ascontiguousarray(info[:, 0]).tobytes()
