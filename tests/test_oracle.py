"""Pins for the CPU oracle: every oracle routine is checked against something
other than itself - numbers the paper prints, closed forms, library routines
(torch.optim in float64, numpy norms, torch's bf16 cast), brute force on tiny
inputs, and the invariants the paper states (sharded == unsharded, pads never
leak, pack/unpack is the identity)."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import ws_oracle as O
from paper_2004_13336_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
RS = [1, 2, 3, 4, 7, 8, 10, 16, 64, 1024]


def _hyper(opt, **kw):
    h = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0, momentum=0.0,
             grad_scale=1.0, step=10)
    h.update(kw)
    return O.make_hyper(opt, h), h


def _rand_model(rng, numels, R, gstd=1e-2, bf16=False):
    w = [rng.normal(0, 0.02, n).astype(np.float32) for n in numels]
    m = [rng.normal(0, 1e-3, n).astype(np.float32) for n in numels]
    v = [np.abs(rng.normal(0, 1e-5, n)).astype(np.float32) for n in numels]
    g = [[rng.normal(0, gstd, n).astype(np.float32) for n in numels] for _ in range(R)]
    if bf16:
        g = [[O.f32_to_bf16_bits(x) for x in gk] for gk in g]
    return w, m, v, g


# ----------------------------------------------------------------- plan ----
def _golden_rows():
    rows = []
    with open(os.path.join(GOLDEN, "plan_worked.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            rows.append([c.strip() for c in line.split("|")])
    return rows


@pytest.mark.parametrize("row", _golden_rows(), ids=lambda r: r[0])
@pytest.mark.parametrize("A", [8, 32])
def test_plan_paper_worked_numbers(row, A):
    name, numel, R, piece, pad, max_total, _where = row
    p = O.Plan([int(numel)], int(R), A)
    if piece != "-":
        assert p.piece[0] == int(piece)
        assert p.R * p.piece[0] - int(numel) == int(pad)
    assert p.R * p.piece[0] <= int(max_total)
    assert p.S == p.piece[0]


def test_plan_two_kb_shard_bytes():
    # Section 5.2: 4 MB / 2048 = 2 KB
    p = O.Plan([4 * 1024 * 1024 // 4], 2048, 8)
    assert p.piece[0] * 4 == 2048


@pytest.mark.parametrize("R", RS)
@pytest.mark.parametrize("A", [8, 32, 128])
def test_plan_closed_forms(R, A):
    rng = np.random.default_rng(R * 1000 + A)
    numel = [1, 2, 7, 31, 64, 997, 1024, 4099] + list(rng.integers(1, 50000, 12))
    p = O.Plan(numel, R, A)
    assert (p.piece % A == 0).all() and (p.piece > 0).all()
    assert (R * p.piece >= p.numel).all()                # every element has a home
    assert (R * p.piece - p.numel < R * A).all()         # padding bound
    assert p.off[0] == 0
    assert (np.diff(p.off) == p.piece[:-1]).all()        # pieces back to back
    assert p.S == p.piece.sum() and p.S * R >= p.N


@pytest.mark.parametrize("R,A", [(1, 8), (3, 8), (4, 16), (7, 8), (16, 8)])
def test_plan_map_is_a_bijection_onto_valid_positions(R, A):
    # brute force: enumerate every (t, i), the location in [R][S] is unique,
    # and every position not hit is a pad.
    numel = [1, 5, 8, 9, 63, 64, 65, 130]
    p = O.Plan(numel, R, A)
    hit = {}
    for t, n in enumerate(numel):
        for i in range(n):
            r, q = divmod(i, int(p.piece[t]))
            assert r < R
            pos = r * p.S + int(p.off[t]) + q
            assert pos not in hit
            hit[pos] = (t, i)
    assert len(hit) == sum(numel)
    assert max(hit) < p.G


def test_plan_workload_shard_lengths():
    # shard lengths of the five model-shaped workloads at A=32
    cases = [(W.tiny(), 11488), (W.resnet50(), 3195232), (W.transformer(128), 1648736),
             (W.transformer(1024), 208576), (W.bert_large(), 20946368),
             (W.decoder_1p5b(), 389408224)]
    for wl, S in cases:
        assert O.Plan(wl.numels, wl.R, 32).S == S, wl.name
    assert O.Plan(W.transformer(1024).numels, 1024, 8).S == 206448
    for R in (1, 2, 8, 32):
        assert O.Plan(W.transformer(R).numels, R, 32).S * R == W.transformer(R).N


# -------------------------------------------------------- pack / unpack ----
def _py_pack(numel, piece, off, S, R, tensors, dtype):
    flat = np.zeros(R * S, dtype=dtype)
    for r in range(R):
        for t in range(len(numel)):
            for q in range(int(piece[t])):
                loc = r * int(piece[t]) + q
                if loc < numel[t]:
                    flat[r * S + int(off[t]) + q] = tensors[t][loc]
    return flat


@pytest.mark.parametrize("R", [1, 2, 3, 7, 16])
@pytest.mark.parametrize("dtype", [np.float32, np.uint16])
def test_pack_matches_definition_bruteforce(R, dtype):
    rng = np.random.default_rng(R)
    numel = [1, 3, 17, 64, 100]
    p = O.Plan(numel, R, 8)
    if dtype == np.float32:
        tensors = [rng.normal(size=n).astype(np.float32) for n in numel]
    else:
        tensors = [rng.integers(1, 65535, n).astype(np.uint16) for n in numel]
    flat = O.pack(p, tensors)
    ref = _py_pack(numel, p.piece, p.off, p.S, R, tensors, dtype)
    assert flat.tobytes() == ref.tobytes()


@pytest.mark.parametrize("R", RS)
@pytest.mark.parametrize("dtype", [np.float32, np.uint16])
def test_pack_unpack_identity_and_zero_pads(R, dtype):
    rng = np.random.default_rng(R + 5)
    numel = [1, 2, 13, 127, 128, 1031, 4096, 9973]          # n < R, n = 1, n prime
    p = O.Plan(numel, R, 8)
    bits = np.uint32 if dtype == np.float32 else np.uint16
    tensors = [rng.integers(1, np.iinfo(bits).max, n, dtype=np.uint64).astype(bits).view(dtype)
               for n in numel]
    flat = O.pack(p, tensors)
    back = O.unpack(p, flat)
    for a, b in zip(tensors, back):
        assert a.tobytes() == b.tobytes()
    # all inputs have non-zero bits, so zero bits are exactly the pads
    assert int((flat.view(bits) == 0).sum()) == p.G - p.N


# --------------------------------------------------------------- reduce ----
@pytest.mark.parametrize("R", [1, 2, 8, 33])
@pytest.mark.parametrize("bf16", [False, True])
def test_reduce_exact_on_integers(R, bf16):
    numel = [5, 64, 300]
    p = O.Plan(numel, R, 8)
    rng = np.random.default_rng(1)
    g = [[rng.integers(-64, 64, n).astype(np.float32) for n in numel] for _ in range(R)]
    expect = [sum(gk[t].astype(np.int64) for gk in g) for t in range(len(numel))]
    if bf16:
        g = [[O.f32_to_bf16_bits(x) for x in gk] for gk in g]
    packed = [O.pack(p, gk) for gk in g]
    red = np.concatenate([O.shard_reduce(p, r, packed) for r in range(R)])
    got = O.unpack(p, red)
    for a, b in zip(got, expect):
        assert (a.astype(np.int64) == b).all()


def test_reduce_arithmetic_series_and_scale():
    R, numel = 16, [40, 9]
    p = O.Plan(numel, R, 8)
    packed = [O.pack(p, [np.full(n, float(k), np.float32) for n in numel]) for k in range(R)]
    for r in range(R):
        red = O.shard_reduce(p, r, packed, grad_scale=0.5)
        full = np.zeros(p.G, np.float32)
        full[r * p.S:(r + 1) * p.S] = red
        for t, x in enumerate(O.unpack(p, full)):
            lo, hi = r * int(p.piece[t]), min(numel[t], (r + 1) * int(p.piece[t]))
            assert (x[lo:hi] == 0.5 * R * (R - 1) / 2).all()


# -------------------------------------- SGD / Adam vs torch.optim (R = 1) ----
def _torch_step(kind, h, w, m, v, g):
    p = torch.nn.Parameter(torch.tensor(w, dtype=torch.float64))
    if kind == "sgdm":
        opt = torch.optim.SGD([p], lr=h["lr"], momentum=h["momentum"],
                              weight_decay=h["weight_decay"])
        opt.state[p]["momentum_buffer"] = torch.tensor(m, dtype=torch.float64)
    else:
        cls = torch.optim.AdamW if kind == "adamw" else torch.optim.Adam
        opt = cls([p], lr=h["lr"], betas=(h["beta1"], h["beta2"]), eps=h["eps"],
                  weight_decay=h["weight_decay"] if kind == "adamw" else 0.0)
        opt.state[p]["step"] = torch.tensor(float(h["step"] - 1))
        opt.state[p]["exp_avg"] = torch.tensor(m, dtype=torch.float64)
        opt.state[p]["exp_avg_sq"] = torch.tensor(v, dtype=torch.float64)
    p.grad = torch.tensor(g, dtype=torch.float64)
    opt.step()
    st = opt.state[p]
    if kind == "sgdm":
        return p.detach().numpy(), st["momentum_buffer"].numpy(), None
    return p.detach().numpy(), st["exp_avg"].numpy(), st["exp_avg_sq"].numpy()


@pytest.mark.parametrize("R", [1, 4])
@pytest.mark.parametrize("step", [1, 10, 1000])
def test_adam_matches_torch_optim_float64(R, step):
    rng = np.random.default_rng(step + R)
    n = 4099
    hs, h = _hyper("adam", step=step)
    w, m, v, g = _rand_model(rng, [n], R)
    gsum = sum(gk[0].astype(np.float64) for gk in g)
    tw, tm, tv = _torch_step("adam", h, w[0], m[0], v[0], gsum)
    O.update_tensor(hs, [gk[0] for gk in g], w[0], m[0], v[0])
    assert (w[0] == tw.astype(np.float32)).mean() > 0.999      # same value up to double rounding
    np.testing.assert_allclose(w[0], tw, rtol=2e-7, atol=0)
    np.testing.assert_allclose(m[0], tm, rtol=2e-7, atol=0)
    np.testing.assert_allclose(v[0], tv, rtol=2e-7, atol=0)


@pytest.mark.parametrize("R", [1, 8])
def test_sgdm_matches_torch_optim_float64(R):
    rng = np.random.default_rng(R)
    n = 5001
    hs, h = _hyper("sgdm", lr=0.1, momentum=0.9, weight_decay=5e-5)
    w, m, _, g = _rand_model(rng, [n], R, gstd=1e-3)
    gsum = sum(gk[0].astype(np.float64) for gk in g)
    tw, tm, _ = _torch_step("sgdm", h, w[0], m[0], None, gsum)
    O.update_tensor(hs, [gk[0] for gk in g], w[0], m[0], None)
    np.testing.assert_allclose(w[0], tw, rtol=2e-7, atol=0)
    np.testing.assert_allclose(m[0], tm, rtol=2e-7, atol=0)


def test_adam_and_sgd_closed_forms():
    rng = np.random.default_rng(0)
    n = 1000
    w0 = rng.normal(0, 0.02, n).astype(np.float32)
    g = rng.normal(0, 1e-2, n).astype(np.float32)
    # Adam, zero slots, first step: w' = w - lr * g / (|g| + eps)
    hs, h = _hyper("adam", step=1)
    w, m, v = w0.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32)
    O.update_tensor(hs, [g], w, m, v)
    gd = g.astype(np.float64)
    np.testing.assert_allclose(w, w0 - h["lr"] * gd / (np.abs(gd) + h["eps"]), rtol=1e-7)
    # plain SGD: w' = w - lr * g
    hs, h = _hyper("sgdm", lr=0.5)
    w, m = w0.copy(), np.zeros(n, np.float32)
    O.update_tensor(hs, [g], w, m, None)
    np.testing.assert_array_equal(w, (w0.astype(np.float64) - 0.5 * gd).astype(np.float32))
    np.testing.assert_array_equal(m, g)
    # zero gradient: weights stay, first moment decays by beta1 / momentum
    hs, h = _hyper("adam")
    m0 = rng.normal(0, 1e-3, n).astype(np.float32)
    w, m, v = w0.copy(), m0.copy(), np.zeros(n, np.float32)
    O.update_tensor(hs, [np.zeros(n, np.float32)], w, m, v)
    np.testing.assert_array_equal(m, (0.9 * m0.astype(np.float64)).astype(np.float32))
    # grad_scale = 1/R turns the sum into the mean
    hs, h = _hyper("sgdm", lr=1.0, grad_scale=0.25)
    w, m = np.zeros(n, np.float32), np.zeros(n, np.float32)
    O.update_tensor(hs, [g, g, g, g], w, m, None)
    np.testing.assert_array_equal(w, -g)


# ----------------------------------------------------------------- LAMB ----
@pytest.mark.parametrize("wd", [0.0, 0.01])
@pytest.mark.parametrize("R", [1, 4])
def test_lamb_from_adamw_direction_and_numpy_norms(wd, R):
    # u = (w - w'_AdamW) / lr (decoupled decay), rho = ||w|| / ||u|| via library routines
    rng = np.random.default_rng(7)
    n = 3001
    hs, h = _hyper("lamb", eps=1e-6, weight_decay=wd)
    w, m, v, g = _rand_model(rng, [n], R)
    w0 = w[0].astype(np.float64)
    gsum = sum(gk[0].astype(np.float64) for gk in g)
    tw, tm, tv = _torch_step("adamw", h, w[0], m[0], v[0], gsum)
    u = (w0 - tw) / h["lr"]
    rho_ref = np.linalg.norm(w0) / np.linalg.norm(u)
    rho = O.update_tensor(hs, [gk[0] for gk in g], w[0], m[0], v[0])
    assert abs(rho - rho_ref) / rho_ref < 1e-9
    np.testing.assert_allclose(w[0], w0 - h["lr"] * rho_ref * u, rtol=3e-7, atol=1e-12)
    np.testing.assert_allclose(m[0], tm, rtol=2e-7)
    np.testing.assert_allclose(v[0], tv, rtol=2e-7)


def test_lamb_closed_forms():
    n = 512
    rng = np.random.default_rng(3)
    # zero slots, step 1, no decay: u = g/(|g|+eps) ~ sign(g); rho = RMS(w)
    hs, h = _hyper("lamb", eps=1e-12, step=1)
    w0 = rng.normal(0, 0.02, n).astype(np.float32)
    g = rng.normal(0, 1e-2, n).astype(np.float32)
    w, m, v = w0.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32)
    rho = O.update_tensor(hs, [g], w, m, v)
    rms = math.sqrt(float((w0.astype(np.float64) ** 2).mean()))
    assert abs(rho - rms) / rms < 1e-6
    np.testing.assert_allclose(w, w0 - h["lr"] * rms * np.sign(g), rtol=1e-5, atol=1e-10)
    # constant tensors: rho = |c| / |u| exactly
    hs, h = _hyper("lamb", eps=1e-6, weight_decay=0.01)
    c, d = 0.5, 0.25
    w, m, v = (np.full(n, c, np.float32), np.zeros(n, np.float32), np.zeros(n, np.float32))
    rho = O.update_tensor(hs, [np.full(n, d, np.float32)], w, m, v)
    bc1, bc2 = 1 - 0.9 ** 10, 1 - 0.999 ** 10
    u = (0.1 * d / bc1) / (math.sqrt(0.001 * d * d / bc2) + 1e-6) + 0.01 * c
    assert abs(rho - c / abs(u)) < 1e-12
    np.testing.assert_allclose(w, c - h["lr"] * (c / abs(u)) * u, rtol=1e-7)
    # zero weight norm or zero update norm -> rho = 1
    hs, h = _hyper("lamb", eps=1e-6)
    w, m, v = (np.zeros(n, np.float32), np.zeros(n, np.float32), np.zeros(n, np.float32))
    assert O.update_tensor(hs, [g], w, m, v) == 1.0
    w, m, v = (w0.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32))
    assert O.update_tensor(hs, [np.zeros(n, np.float32)], w, m, v) == 1.0
    np.testing.assert_array_equal(w, w0)


def test_lamb_trust_ratio_scales_with_weights():
    rng = np.random.default_rng(11)
    n = 777
    hs, _ = _hyper("lamb", eps=1e-6)
    w, m, v, g = _rand_model(rng, [n], 2)
    r1 = O.update_tensor(hs, [gk[0] for gk in g], w[0].copy(), m[0].copy(), v[0].copy())
    r4 = O.update_tensor(hs, [gk[0] for gk in g], (4 * w[0]).copy(), m[0].copy(), v[0].copy())
    assert abs(r4 / r1 - 4.0) < 1e-12


# ------------------------------------------------- sharded == unsharded ----
def _run_both(opt, R, A, numel, bf16=False, poison=False, out_dtype=None, seed=0, **hk):
    rng = np.random.default_rng(seed)
    hs, h = _hyper(opt, **hk)
    w, m, v, g = _rand_model(rng, numel, R, bf16=bf16)
    p = O.Plan(numel, R, A)
    pw, pm, pv = O.pack(p, w), O.pack(p, m), O.pack(p, v)
    pg = [O.pack(p, gk) for gk in g]
    if poison:
        valid = O.pack(p, [np.ones(n, np.float32) for n in numel]) != 0
        nanbits = np.float32(np.nan)
        for buf in (pw, pm, pv):
            buf[~valid] = nanbits
        for buf in pg:
            if buf.dtype == np.uint16:
                buf[~valid] = 0x7FC0
            else:
                buf[~valid] = nanbits
    uw, um, uv = [x.copy() for x in w], [x.copy() for x in m], [x.copy() for x in v]
    has_v = opt in ("adam", "lamb")
    rho_u = O.update_unsharded(hs, g, uw, um, uv if has_v else None)
    gathered, rho_s, partials = O.sharded_update(hs, p, pg, pw, pm, pv if has_v else None,
                                                 out_dtype)
    return p, (uw, um, uv, rho_u), (pw, pm, pv, gathered, rho_s, partials)


@pytest.mark.parametrize("opt", ["sgdm", "adam"])
@pytest.mark.parametrize("R", RS)
def test_sharded_equals_unsharded_bit_identical(opt, R):
    numel = [1, 9, 64, 333, 2048, 5000]
    p, (uw, um, uv, _), (pw, pm, pv, _, _, _) = _run_both(
        opt, R, 8, numel, momentum=0.9, weight_decay=5e-5 if opt == "sgdm" else 0.0, seed=R)
    for a, b in zip(uw, O.unpack(p, pw)):
        assert a.tobytes() == b.tobytes()
    for a, b in zip(um, O.unpack(p, pm)):
        assert a.tobytes() == b.tobytes()
    if opt == "adam":
        for a, b in zip(uv, O.unpack(p, pv)):
            assert a.tobytes() == b.tobytes()


@pytest.mark.parametrize("opt", ["sgdm", "adam", "lamb"])
def test_thread_count_does_not_change_any_bit(opt):
    # the all-core timing of the benchmark runs the same code on more threads: only loops with
    # independent iterations are split, every sum keeps its one fixed order
    numel = [1, 9, 64, 333, 2048, 5000, 70001, 300000]      # large enough for the loops to go parallel
    prev = O.set_num_threads(1)
    try:
        _, _, one = _run_both(opt, 7, 8, numel, momentum=0.9, weight_decay=0.01, bf16=(opt == "adam"), seed=3,
                              out_dtype=O.BF16)
        O.set_num_threads(max(2, os.cpu_count() or 2))
        assert O.num_threads() >= 2
        _, _, many = _run_both(opt, 7, 8, numel, momentum=0.9, weight_decay=0.01, bf16=(opt == "adam"), seed=3,
                               out_dtype=O.BF16)
    finally:
        O.set_num_threads(prev)
    for a, b in zip(one, many):
        if a is not None:
            assert np.asarray(a).tobytes() == np.asarray(b).tobytes()


@pytest.mark.parametrize("opt", ["lamb", "lars"])
@pytest.mark.parametrize("R", [1, 3, 8])
def test_one_replicas_phases_compose_to_the_sharded_update(opt, R):
    # Section 4.1: every replica reduces what its shard holds, the partial results are combined, then
    # every replica applies.  The per-replica phase functions, run for r = 0..R-1 around a sum of the
    # partials in ascending r, must give bit for bit what the all-shard routine gives (one gradient copy:
    # the reduce-scatter has already summed the replicas' copies).
    rng = np.random.default_rng(40 + R)
    numel = [1, 9, 64, 333, 2048, 5000]
    hs, _ = _hyper(opt, momentum=0.9, weight_decay=0.01, trust_coeff=0.02, lr=0.5 if opt == "lars" else 1e-3)
    w, m, v, g = _rand_model(rng, numel, 1)
    p = O.Plan(numel, R, 8)
    pw, pm, pv, pg = O.pack(p, w), O.pack(p, m), O.pack(p, v), O.pack(p, g[0])
    aw, am, av = pw.copy(), pm.copy(), pv.copy()
    gathered, rho, _ = O.sharded_update(hs, p, [pg], aw, am, av if opt == "lamb" else None, O.BF16)
    S = p.S
    parts, us = [], []
    for r in range(R):
        sl = slice(r * S, (r + 1) * S)
        part, u = O.norm_shard_partial(hs, p, r, pg[sl], pw[sl], pm[sl], pv[sl] if opt == "lamb" else None)
        parts.append(part)
        us.append(u)
    tot = np.zeros((p.T, 2))
    for part in parts:                       # ascending r
        tot += part
    ratio = np.array([O.norm_ratio(hs, a, b) for a, b in tot])
    assert ratio.tobytes() == np.asarray(rho).tobytes()
    slots = [O.norm_shard_apply(hs, p, r, ratio, us[r], pw[r * S:(r + 1) * S], pm[r * S:(r + 1) * S], O.BF16)
             for r in range(R)]
    assert pw.tobytes() == aw.tobytes() and pm.tobytes() == am.tobytes()
    if opt == "lamb":
        assert pv.tobytes() == av.tobytes()
    assert np.concatenate(slots).tobytes() == gathered.tobytes()


@pytest.mark.parametrize("R", [1, 3, 8, 64])
@pytest.mark.parametrize("bf16", [False, True])
def test_sharded_lamb_equals_unsharded_within_one_ulp(R, bf16):
    numel = [1, 9, 64, 333, 2048, 5000]           # tensors inside one shard and across all
    p, (uw, um, uv, rho_u), (pw, pm, pv, _, rho_s, partials) = _run_both(
        "lamb", R, 8, numel, bf16=bf16, eps=1e-6, weight_decay=0.01, seed=R)
    np.testing.assert_allclose(rho_s, rho_u, rtol=1e-13)
    for a, b in zip(uw, O.unpack(p, pw)):
        ulp = np.spacing(np.abs(a))
        assert (np.abs(a.astype(np.float64) - b) <= ulp).all()
    for a, b in zip(um, O.unpack(p, pm)):
        assert a.tobytes() == b.tobytes()
    # a tensor with n_t <= p_t lives in shard 0 only: higher shards contribute nothing
    for t, n in enumerate(numel):
        for r in range(R):
            if r * int(p.piece[t]) >= n:
                assert partials[r, t, 0] == 0.0 and partials[r, t, 1] == 0.0


@pytest.mark.parametrize("opt", ["sgdm", "adam", "lamb"])
@pytest.mark.parametrize("bf16", [False, True])
def test_poisoned_pads_never_leak(opt, bf16):
    numel = [1, 9, 64, 333, 2050]
    kw = dict(momentum=0.9, weight_decay=0.01, eps=1e-6)
    p, _, clean = _run_both(opt, 7, 32, numel, bf16=bf16, out_dtype=O.BF16, seed=1, **kw)
    _, _, dirty = _run_both(opt, 7, 32, numel, bf16=bf16, out_dtype=O.BF16, seed=1, poison=True, **kw)
    used = [0, 1, 3] if opt == "sgdm" else [0, 1, 2, 3]     # (w, m, v, gathered); SGD has no v
    for i in used:
        assert clean[i].tobytes() == dirty[i].tobytes()
    np.testing.assert_array_equal(clean[4], dirty[4])
    valid = O.pack(p, [np.ones(n, np.float32) for n in numel]) != 0
    for buf in [dirty[i] for i in used[:-1]]:
        assert (buf.view(np.uint32)[~valid] == 0).all()         # output pads are +0
    assert (dirty[3][~valid] == 0).all()


# ------------------------------------------------------------------ bf16 ----
def test_bf16_rounding_matches_torch_and_edge_table():
    rng = np.random.default_rng(2)
    x = np.concatenate([rng.normal(0, 1, 4000), rng.normal(0, 1e-30, 500),
                        rng.normal(0, 1e30, 500)]).astype(np.float32)
    bits = O.f32_to_bf16_bits(x)
    tb = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(bits, tb)
    def f(u):
        return np.array([u], dtype=np.uint32).view(np.float32)[0]
    table = [
        (f(0x3F808000), 0x3F80),   # tie, even stays
        (f(0x3F818000), 0x3F82),   # tie, odd rounds up to even
        (f(0x3F808001), 0x3F81),   # just above tie
        (f(0x3F807FFF), 0x3F80),   # just below tie
        (f(0x00000000), 0x0000), (f(0x80000000), 0x8000),   # signed zeros
        (f(0x7F7FFFFF), 0x7F80),   # max finite fp32 rounds to +inf in bf16
        (f(0x7F7F0000), 0x7F7F),   # max finite bf16
        (f(0x00008000), 0x0000),   # subnormal tie to even (0)
        (f(0x00018000), 0x0002),   # subnormal tie to even (up)
        (f(0x7F800000), 0x7F80), (f(0xFF800000), 0xFF80),   # infinities
    ]
    for val, want in table:
        assert int(O.f32_to_bf16_bits(np.array([val]))[0]) == want
    assert np.isnan(O.bf16_bits_to_f64(O.f32_to_bf16_bits(np.array([np.nan], np.float32))))[0]
    # widening is exact
    np.testing.assert_array_equal(O.bf16_bits_to_f64(bits),
                                  torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).double().numpy())


def test_gathered_bf16_is_rne_of_fp32_master():
    numel = [9, 64, 333]
    p, _, (pw, _, _, gathered, _, _) = _run_both("adam", 4, 8, numel, out_dtype=O.BF16)
    tb = torch.from_numpy(pw).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(gathered, tb)


def test_tiny_workload_end_to_end():
    # config "tiny" through the workload generators: both oracle routes agree
    wl = W.tiny()
    hs = O.make_hyper(wl.opt, wl.hyper)
    w, m, v = [[x.numpy() for x in lst] for lst in W.make_state(wl)]
    g = [[x.numpy() for x in gk] for gk in W.make_grads(wl)]
    p = O.Plan(wl.numels, wl.R, 32)
    pw, pm, pv = O.pack(p, w), O.pack(p, m), O.pack(p, v)
    O.sharded_update(hs, p, [O.pack(p, gk) for gk in g], pw, pm, pv)
    O.update_unsharded(hs, g, w, m, v)
    for a, b in zip(w, O.unpack(p, pw)):
        assert a.tobytes() == b.tobytes()


def test_empty_tensors_are_inert():
    # an empty tensor has no piece; the model around it updates exactly as without it
    numel_a, numel_b = [40, 0, 333, 0, 9], [40, 333, 9]
    outs = []
    for numel in (numel_a, numel_b):
        p, (uw, um, uv, rho_u), (pw, pm, pv, _, rho_s, _) = _run_both("lamb", 4, 8, numel, eps=1e-6,
                                                                       weight_decay=0.01, seed=3)
        outs.append((p, [x for x in O.unpack(p, pw) if x.size], [r for r, n in zip(rho_s, numel) if n]))
        for r, n in zip(rho_s, numel):
            if n == 0:
                assert r == 1.0
    assert outs[0][0].S == outs[1][0].S
    # same seeds draw different streams for different tensor lists, so compare structure only
    assert [x.size for x in outs[0][1]] == [x.size for x in outs[1][1]]
    flat = O.pack(outs[0][0], [np.arange(n, dtype=np.float32) + 1 for n in numel_a])
    back = O.unpack(outs[0][0], flat)
    assert [b.size for b in back] == numel_a and (back[2] == np.arange(333) + 1).all()


@pytest.mark.parametrize("groups,M", [(2, 4), (4, 2), (3, 1), (1, 5)])
def test_partial_sharding_equals_unsharded(groups, M):
    # Section 5.2: N groups of M replicas, each group shards M ways; the cross-group all-reduce
    # adds the groups' partial shards -> shard j holds the sum of all N*M gradient copies
    numel = [9, 64, 333, 2048]
    K = groups * M
    rng = np.random.default_rng(K)
    hs, _ = _hyper("adam")
    w, m, v, g = _rand_model(rng, numel, K)
    p = O.Plan(numel, M, 8)
    pw, pm, pv = O.pack(p, w), O.pack(p, m), O.pack(p, v)
    O.sharded_update(hs, p, [O.pack(p, gk) for gk in g], pw, pm, pv)
    O.update_unsharded(hs, g, w, m, v)
    for a, b in zip(w, O.unpack(p, pw)):
        assert a.tobytes() == b.tobytes()
    for a, b in zip(v, O.unpack(p, pv)):
        assert a.tobytes() == b.tobytes()


# ----------------------------------------------------------------- LARS ----
def _lars_hyper(**kw):
    h = dict(lr=10.0, beta1=0.0, beta2=0.0, eps=0.0, weight_decay=5e-5, momentum=0.9, grad_scale=1.0,
             step=1, trust_coeff=0.001)
    h.update(kw)
    return O.make_hyper("lars", h), h


@pytest.mark.parametrize("K", [1, 8])
def test_lars_from_torch_sgd_with_local_rate_and_numpy_norms(K):
    # with lambda = eta ||w|| / (||g|| + beta ||w||) from library norms, one LARS step is one
    # torch.optim.SGD step at lr*lambda whose momentum buffer is v / (lr*lambda)
    rng = np.random.default_rng(K)
    n = 2501
    hs, h = _lars_hyper()
    w, m, _, g = _rand_model(rng, [n], K, gstd=1e-3)
    w0, v0 = w[0].astype(np.float64), m[0].astype(np.float64)
    gsum = sum(gk[0].astype(np.float64) for gk in g)
    lam = h["trust_coeff"] * np.linalg.norm(w0) / (np.linalg.norm(gsum) + h["weight_decay"] * np.linalg.norm(w0))
    eff = h["lr"] * lam
    p = torch.nn.Parameter(torch.tensor(w0))
    opt = torch.optim.SGD([p], lr=eff, momentum=h["momentum"], weight_decay=h["weight_decay"])
    opt.state[p]["momentum_buffer"] = torch.tensor(v0 / eff)
    p.grad = torch.tensor(gsum)
    opt.step()
    rate = O.update_tensor(hs, [gk[0] for gk in g], w[0], m[0], None)
    assert abs(rate - lam) / lam < 1e-12
    np.testing.assert_allclose(w[0], p.detach().numpy(), rtol=2e-7, atol=1e-12)
    np.testing.assert_allclose(m[0], eff * opt.state[p]["momentum_buffer"].numpy(), rtol=2e-7, atol=1e-14)


def test_lars_closed_forms():
    n = 400
    rng = np.random.default_rng(5)
    w0 = rng.normal(0, 0.02, n).astype(np.float32)
    g = rng.normal(0, 1e-3, n).astype(np.float32)
    # no decay, no momentum: the step length lr*eta*||w|| does not depend on the gradient's scale
    hs, h = _lars_hyper(weight_decay=0.0, momentum=0.0)
    outs = []
    for scale in (1.0, 64.0):
        w, m = w0.copy(), np.zeros(n, np.float32)
        O.update_tensor(hs, [(g * scale).astype(np.float32)], w, m, None)
        outs.append(w)
        step = np.linalg.norm(w.astype(np.float64) - w0)
        expect = h["lr"] * h["trust_coeff"] * np.linalg.norm(w0.astype(np.float64))
        assert abs(step - expect) / expect < 1e-5
    np.testing.assert_allclose(outs[0], outs[1], rtol=1e-6)
    # constant tensors: lambda = eta c / (d + beta c)
    hs, h = _lars_hyper()
    c, d = 0.5, 0.25
    w, m = np.full(n, c, np.float32), np.zeros(n, np.float32)
    rate = O.update_tensor(hs, [np.full(n, d, np.float32)], w, m, None)
    lam = 0.001 * c / (d + 5e-5 * c)
    assert abs(rate - lam) < 1e-15
    np.testing.assert_allclose(w, c - 10.0 * lam * (d + 5e-5 * c), rtol=1e-7)
    # zero weight norm or zero gradient norm: local rate 1
    w, m = np.zeros(n, np.float32), np.zeros(n, np.float32)
    assert O.update_tensor(hs, [g], w, m, None) == 1.0
    w, m = w0.copy(), np.zeros(n, np.float32)
    assert O.update_tensor(hs, [np.zeros(n, np.float32)], w, m, None) == 1.0


@pytest.mark.parametrize("R", [1, 3, 8, 64])
@pytest.mark.parametrize("bf16", [False, True])
def test_sharded_lars_equals_unsharded_within_one_ulp(R, bf16):
    numel = [1, 9, 64, 333, 2048, 5000]
    p, (uw, um, _, rate_u), (pw, pm, _, gathered, rate_s, _) = _run_both(
        "lars", R, 8, numel, bf16=bf16, out_dtype=O.BF16, seed=R, lr=10.0, momentum=0.9, weight_decay=5e-5,
        trust_coeff=0.001)
    np.testing.assert_allclose(rate_s, rate_u, rtol=1e-13)
    for a, b in zip(uw, O.unpack(p, pw)):
        assert (np.abs(a.astype(np.float64) - b) <= np.spacing(np.abs(a))).all()
    for a, b in zip(um, O.unpack(p, pm)):
        assert (np.abs(a.astype(np.float64) - b) <= np.spacing(np.abs(a))).all()
    np.testing.assert_array_equal(gathered, O.f32_to_bf16_bits(pw))


def test_lars_poisoned_pads_never_leak():
    numel = [1, 9, 64, 333, 2050]
    kw = dict(lr=10.0, momentum=0.9, weight_decay=5e-5, trust_coeff=0.001)
    p, _, clean = _run_both("lars", 7, 32, numel, out_dtype=O.BF16, seed=1, **kw)
    _, _, dirty = _run_both("lars", 7, 32, numel, out_dtype=O.BF16, seed=1, poison=True, **kw)
    for i in (0, 1, 3):
        assert clean[i].tobytes() == dirty[i].tobytes()
    np.testing.assert_array_equal(clean[4], dirty[4])


# ------------------------------------------- concatenated (flat) layout ----
@pytest.mark.parametrize("R", [1, 3, 8, 64, 1024])
@pytest.mark.parametrize("A", [8, 32])
def test_flat_plan_partitions_the_concatenation(R, A):
    numel = [1, 5, 8, 9, 63, 64, 65, 130, 0, 4099]
    p = O.FlatPlan(numel, R, A)
    assert p.cat[0] == 0 and (p.cat % A == 0).all()
    assert (np.diff(p.cat) >= p.numel).all() and (np.diff(p.cat) - p.numel < A).all()   # only alignment gaps
    assert p.S % A == 0 and p.G >= p.cat[-1] and p.G - p.cat[-1] < R * A                # and a short tail
    tmap = p.tensor_map()
    assert int((tmap >= 0).sum()) == sum(numel)
    for t, n in enumerate(numel):                       # every element has exactly one position, in order
        assert (np.nonzero(tmap == t)[0] == p.cat[t] + np.arange(n)).all()
    # never more padding than the per-tensor layout
    assert p.G <= O.Plan(numel, R, A).G


def test_flat_layout_has_almost_no_padding_at_1024_shards():
    wl = W.transformer(1024)
    flat, per = O.FlatPlan(wl.numels, 1024, 32), O.Plan(wl.numels, 1024, 32)
    assert flat.G - wl.N < 40000 and per.G - wl.N > 2_000_000


@pytest.mark.parametrize("R", [1, 2, 3, 7, 16])
@pytest.mark.parametrize("dtype", [np.float32, np.uint16])
def test_flat_pack_unpack_identity(R, dtype):
    rng = np.random.default_rng(R)
    numel = [1, 2, 13, 127, 128, 1031, 4096]
    p = O.FlatPlan(numel, R, 8)
    bits = np.uint32 if dtype == np.float32 else np.uint16
    tensors = [rng.integers(1, np.iinfo(bits).max, n, dtype=np.uint64).astype(bits).view(dtype) for n in numel]
    flat = O.pack_flat(p, tensors)
    for a, b in zip(tensors, O.unpack_flat(p, flat)):
        assert a.tobytes() == b.tobytes()
    assert int((flat.view(bits) == 0).sum()) == p.G - p.N


@pytest.mark.parametrize("opt", ["sgdm", "adam", "lamb", "lars"])
@pytest.mark.parametrize("R", [1, 3, 8, 64])
def test_flat_sharded_equals_unsharded(opt, R):
    numel = [1, 9, 64, 333, 2048, 5000]
    rng = np.random.default_rng(R)
    kw = dict(momentum=0.9, weight_decay=5e-5 if opt in ("sgdm", "lars") else (0.01 if opt == "lamb" else 0.0),
              eps=1e-6 if opt == "lamb" else 1e-8, lr=10.0 if opt == "lars" else 1e-3)
    hs, _ = _hyper(opt, **kw)
    w, m, v, g = _rand_model(rng, numel, R, gstd=1e-3)
    has_v = opt in ("adam", "lamb")
    p = O.FlatPlan(numel, R, 8)
    pw, pm, pv = O.pack_flat(p, w), O.pack_flat(p, m), O.pack_flat(p, v)
    valid = p.tensor_map() >= 0
    for buf in (pw, pm, pv):
        buf[~valid] = np.float32(np.nan)                     # pads may hold anything on entry
    pg = [O.pack_flat(p, gk) for gk in g]
    for buf in pg:
        buf[~valid] = np.float32(np.nan)
    gathered, rho_s = O.sharded_update_flat(hs, p, pg, pw, pm, pv if has_v else None, O.BF16)
    rho_u = O.update_unsharded(hs, g, w, m, v if has_v else None)
    np.testing.assert_allclose(rho_s, rho_u, rtol=1e-13)
    exact = opt in ("sgdm", "adam")
    for ref, got in ((w, O.unpack_flat(p, pw)), (m, O.unpack_flat(p, pm))):
        for a, b in zip(ref, got):
            if exact:
                assert a.tobytes() == b.tobytes()
            else:
                assert (np.abs(a.astype(np.float64) - b) <= np.spacing(np.abs(a))).all()
    assert (pw.view(np.uint32)[~valid] == 0).all() and (pm.view(np.uint32)[~valid] == 0).all()
    np.testing.assert_array_equal(gathered, O.f32_to_bf16_bits(pw))


def _tiny_expected():
    rows = {}
    with open(os.path.join(GOLDEN, "tiny_adam_expected.txt")) as f:
        for line in f:
            if line.startswith("#"):
                continue
            p = line.split()
            rows[(p[0], int(p[1]))] = (int(p[2]), float(p[3]), float(p[4]), [float.fromhex(h) for h in p[5:9]])
    return rows


def test_oracle_reproduces_the_stored_tiny_result():
    # regression pin: values written by tests/golden/make_tiny_expected.py (oracle only)
    wl = W.tiny()
    w, m, v = [[x.numpy() for x in lst] for lst in W.make_state(wl, "cpu")]
    g = [[x.numpy() for x in gk] for gk in W.make_grads(wl, "cpu")]
    O.update_unsharded(O.make_hyper(wl.opt, wl.hyper), g, w, m, v)
    rows = _tiny_expected()
    for name, lst in (("w", w), ("m", m), ("v", v)):
        for t, x in enumerate(lst):
            n, s, s2, picks = rows[(name, t)]
            assert x.size == n
            # (a relative tolerance, not bit equality: the CPU random generator's vector maths may
            # differ in the last bit between processor generations)
            rms = np.sqrt(s2 / n)
            assert abs(float((x.astype(np.float64) ** 2).sum()) - s2) <= 1e-6 * s2
            assert abs(float(x.astype(np.float64).sum()) - s) <= 1e-6 * rms * n
            for i, ref in zip((0, n // 3, 2 * n // 3, n - 1), picks):
                assert abs(float(x[i]) - ref) <= 1e-6 * max(abs(ref), rms)
