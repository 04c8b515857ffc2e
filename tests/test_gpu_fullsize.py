"""GPU parity at the full sizes of the five model-shaped workloads, in the
launch configuration the benchmark uses (pack R gradient sets, one fused
update over all shards, unpack).  Where the whole model is too large for the
oracle to finish in seconds, outputs are checked on samples the oracle can
compute one by one: random elements of every tensor plus the elements on both
sides of every shard boundary (momentum-SGD / Adam are elementwise), or whole
tensors (LAMB needs a tensor's norms)."""
import numpy as np
import pytest
import torch

from oracle import ws_oracle as O
from paper_2004_13336_b200 import binding as B
from paper_2004_13336_b200 import workloads as W
from tests._util import TOL_BF16, TOL_FP32, TOL_LAMB, bf16_to_f64, err, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda"
A = 32


def _sample_indices(n, piece, R, rng, k):
    """Random elements plus both sides of every shard boundary and the tensor's ends."""
    idx = [0, n - 1]
    for r in range(1, min(R, 64)):
        b = r * piece
        if b < n:
            idx += [b - 1, b]
    idx += list(rng.integers(0, n, size=min(k, n)))
    return np.unique(np.clip(np.array(idx, dtype=np.int64), 0, n - 1))


def _gather(t, idx_dev):
    return to_np(t[idx_dev])


def _run_sampled(wl, samples_per_tensor=1500, path="unfused", layout="per_tensor"):
    """Elementwise optimizers: full-size GPU step, oracle on sampled elements.
    path "unfused": ws_pack of every gradient list, ws_shard_update, ws_unpack;
    path "fused":   ws_fused_update straight from the gradient lists into weight tensors
                    (the configuration the benchmark reports)."""
    torch.cuda.empty_cache()
    rng = np.random.default_rng(wl.seed)
    plan = B.Plan(wl.shapes, wl.R, A, layout=layout)
    if layout == "concat":
        oplan = O.FlatPlan(wl.numels, wl.R, A)
        # shard boundaries fall inside tensors: sample both sides of the first one in each tensor
        piece = [max(1, int(oplan.S - (oplan.cat[t] % oplan.S))) for t in range(wl.T)]
    else:
        oplan = O.Plan(wl.numels, wl.R, A)
        piece = [int(p) for p in oplan.piece]
    assert (plan.S, plan.N) == (oplan.S, oplan.N)
    idx = [_sample_indices(n, p, wl.R, rng, samples_per_tensor) for n, p in zip(wl.numels, piece)]
    idx_dev = [torch.from_numpy(i).to(DEV) for i in idx]
    w, m, v = W.make_state(wl, DEV)
    sw, sm, sv = ([_gather(x, i) for x, i in zip(lst, idx_dev)] for lst in (w, m, v))
    pw = torch.empty(plan.G, device=DEV)
    pm, pv = torch.empty_like(pw), torch.empty_like(pw)
    for src, dst in ((w, pw), (m, pm), (v, pv)):
        B.ws_pack(plan, src, dst)
    del m, v
    pg, sg, glists = [], [], []
    for k in range(wl.R):
        gk = W.make_grads_one(wl, k, DEV)
        sg.append([_gather(x, i) for x, i in zip(gk, idx_dev)])
        if path == "fused":
            glists.append(gk)
        else:
            b = torch.empty(plan.G, dtype=wl.grad_dtype, device=DEV)
            B.ws_pack(plan, gk, b)
            pg.append(b)
        del gk
    hy = B.make_hyper(wl.opt, wl.hyper)
    gathered = None
    wout = [torch.zeros(n, dtype=wl.out_dtype, device=DEV) for n in wl.numels]
    if path == "fused":
        B.ws_fused_update(plan, -1, B.TensorTable(plan, glists), pw, pm, pv if wl.opt != "sgdm" else None, hy,
                          B.TensorTable(plan, [wout]))
        del glists
    else:
        gathered = torch.empty(plan.G, dtype=wl.out_dtype, device=DEV) if wl.out_dtype != torch.float32 else None
        B.ws_shard_update(plan, -1, pg, pw, pm, pv if wl.opt != "sgdm" else None, hy, gathered)
        B.ws_unpack(plan, gathered if gathered is not None else pw, wout)
        del pg
    # oracle on the sampled elements (each tensor's sample is a small pseudo-tensor)
    hs = O.make_hyper(wl.opt, wl.hyper)
    for t in range(wl.T):
        O.update_tensor(hs, [sg[k][t] for k in range(wl.R)], sw[t], sm[t], sv[t] if wl.opt != "sgdm" else None)
    # GPU outputs back in tensor form
    worst = {"w": 0.0, "m": 0.0, "v": 0.0, "out": 0.0}
    for name, buf, ref in (("w", pw, sw), ("m", pm, sm), ("v", pv, sv)):
        if name == "v" and wl.opt == "sgdm":
            continue
        B.ws_unpack(plan, buf, w)           # reuse the weight tensors as the unpack target
        for t in range(wl.T):
            worst[name] = max(worst[name], err(_gather(w[t], idx_dev[t]), ref[t]))
        if name == "w":                     # the emitted weights: fp32 copy of, or RNE bf16 of, the fp32 master
            for t in range(wl.T):
                assert torch.equal(wout[t], w[t].to(wl.out_dtype)), f"tensor {t}"
    bf = wl.out_dtype == torch.bfloat16
    for t in range(wl.T):
        got = _gather(wout[t], idx_dev[t])
        worst["out"] = max(worst["out"], err(bf16_to_f64(got) if bf else got, sw[t]))
    print(f"{wl.name} R={wl.R} {path}: max err w {worst['w']:.2e} m {worst['m']:.2e} v {worst['v']:.2e} "
          f"out {worst['out']:.2e}")
    assert worst["w"] <= TOL_FP32 and worst["m"] <= TOL_FP32 and worst["v"] <= TOL_FP32
    assert worst["out"] <= (TOL_BF16 if bf else TOL_FP32)
    return worst


def test_resnet50_full_model_every_element():
    """Config 2 whole: 161 tensors, 25.6M params, R=8, momentum-SGD - every element against the oracle."""
    wl = W.resnet50()
    plan = B.Plan(wl.shapes, wl.R, A)
    oplan = O.Plan(wl.numels, wl.R, A)
    w, m, v = W.make_state(wl, DEV)
    g = W.make_grads(wl, DEV)
    ow, om = [to_np(x) for x in w], [to_np(x) for x in m]
    og = [[to_np(x) for x in gk] for gk in g]
    O.update_unsharded(O.make_hyper(wl.opt, wl.hyper), og, ow, om, None)
    pw = torch.empty(plan.G, device=DEV)
    pm = torch.empty_like(pw)
    B.ws_pack(plan, w, pw)
    B.ws_pack(plan, m, pm)
    pg = []
    for gk in g:
        b = torch.empty(plan.G, device=DEV)
        B.ws_pack(plan, gk, b)
        pg.append(b)
    B.ws_shard_update(plan, -1, pg, pw, pm, None, B.make_hyper(wl.opt, wl.hyper))
    outs_w = [torch.empty_like(x) for x in w]
    outs_m = [torch.empty_like(x) for x in w]
    B.ws_unpack(plan, pw, outs_w)
    B.ws_unpack(plan, pm, outs_m)
    ew = max(err(to_np(a), b) for a, b in zip(outs_w, ow))
    em = max(err(to_np(a), b) for a, b in zip(outs_m, om))
    print(f"resnet50 full: err w {ew:.2e} m {em:.2e}")
    assert ew <= TOL_FP32 and em <= TOL_FP32
    # pads of the packed state are +0
    valid = O.pack(oplan, [np.ones(int(n), np.float32) for n in oplan.numel]) != 0
    assert (to_np(pw).view(np.uint32)[~valid] == 0).all() and (to_np(pm).view(np.uint32)[~valid] == 0).all()


@pytest.mark.parametrize("path", ["unfused", "fused"])
@pytest.mark.parametrize("R", [1, 2, 8, 32])
def test_transformer_adam_sampled(R, path):
    _run_sampled(W.transformer(R), path=path)


@pytest.mark.parametrize("path", ["unfused", "fused"])
def test_transformer_adam_R128_sampled(path):
    """108 GB of gradients: the largest replica count that fits one GPU."""
    import gc
    gc.collect()
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < 130e9:
        pytest.skip("needs ~120 GB of free device memory")
    _run_sampled(W.transformer(128), samples_per_tensor=300, path=path)


@pytest.mark.parametrize("path", ["unfused", "fused"])
def test_decoder_1p5b_bf16_grads_bf16_gathered_sampled(path):
    _run_sampled(W.decoder_1p5b(), samples_per_tensor=500, path=path)


@pytest.mark.parametrize("path", ["unfused", "fused"])
@pytest.mark.parametrize("R", [8, 32])
def test_transformer_concat_layout_sampled(R, path):
    """The concatenated layout (Section 5.2) at full size: shards cut tensors wherever they fall."""
    _run_sampled(W.transformer(R), path=path, layout="concat")


def test_resnet50_fused_path_sampled():
    _run_sampled(W.resnet50(), samples_per_tensor=4000, path="fused")


def test_transformer_R1024_window_of_shards():
    """R=1024 cannot hold its 863 GB of gradients; shards are updated one at a time from
    S-element slices (slice mode 1, what a reduce-scatter receive buffer holds).  Window:
    first, second, middle, last and four seeded shards."""
    wl = W.transformer(1024)
    R = wl.R
    plan = B.Plan(wl.shapes, R, A)
    oplan = O.Plan(wl.numels, R, A)
    S = plan.S
    rng = np.random.default_rng(1024)
    window = sorted(set([0, 1, R // 2, R - 1] + list(rng.integers(2, R - 1, 4))))
    hy = B.make_hyper(wl.opt, wl.hyper)
    hs = O.make_hyper(wl.opt, wl.hyper)
    gen = torch.Generator(device=DEV).manual_seed(7)
    gslices = torch.empty(R, S, device=DEV)
    for r in window:
        r = int(r)
        gslices.normal_(0.0, wl.grad_std, generator=gen)
        w = torch.empty(S, device=DEV).normal_(0.0, wl.w_std, generator=gen)
        m = torch.empty(S, device=DEV).normal_(0.0, wl.m_std, generator=gen)
        v = torch.empty(S, device=DEV).normal_(0.0, wl.v_std, generator=gen).abs_()
        gathered = torch.full((plan.G,), 2.0, dtype=torch.bfloat16, device=DEV)
        ow, om, ov = to_np(w), to_np(m), to_np(v)
        og = to_np(gslices)
        # validity of each shard position, from the oracle's plan: location r*p_t + q < n_t
        valid = np.zeros(S, dtype=bool)
        for t in range(oplan.T):
            nv = int(np.clip(oplan.numel[t] - r * oplan.piece[t], 0, oplan.piece[t]))
            valid[int(oplan.off[t]):int(oplan.off[t]) + nv] = True
        O.update_tensor(hs, [og[k] for k in range(R)], ow, om, ov)
        for a in (ow, om, ov):
            a[~valid] = 0.0
        B.ws_shard_update(plan, r, [gslices[k] for k in range(R)], w, m, v, hy, gathered, slice_mode=1)
        for name, got, ref in (("w", w, ow), ("m", m, om), ("v", v, ov)):
            e = err(to_np(got)[valid], ref[valid])
            assert e <= TOL_FP32, f"shard {r} {name}: {e:.3e}"
            assert (to_np(got).view(np.uint32)[~valid] == 0).all()
        assert torch.equal(gathered[r * S:(r + 1) * S], w.to(torch.bfloat16))
        assert bool((gathered[:r * S] == 2.0).all()) and bool((gathered[(r + 1) * S:] == 2.0).all())


def test_bert_large_lamb_whole_tensors():
    """Config 4: LAMB, R=16.  Full-size GPU step; the oracle recomputes whole tensors (their
    norms span all 16 shards): the embedding, the first and last layers, the pooler."""
    wl = W.bert_large()
    torch.cuda.empty_cache()
    plan = B.Plan(wl.shapes, wl.R, A)
    hy = B.make_hyper(wl.opt, wl.hyper)
    hs = O.make_hyper(wl.opt, wl.hyper)
    chosen = sorted(set([0, 1, 2, 3, 4] + list(range(5, 21)) + list(range(wl.T - 18, wl.T))))
    w, m, v = W.make_state(wl, DEV)
    ref = {t: [to_np(w[t]), to_np(m[t]), to_np(v[t])] for t in chosen}
    pw = torch.empty(plan.G, device=DEV)
    pm, pv = torch.empty_like(pw), torch.empty_like(pw)
    for src, dst in ((w, pw), (m, pm), (v, pv)):
        B.ws_pack(plan, src, dst)
    del m, v
    pg, og = [], {t: [] for t in chosen}
    for k in range(wl.R):
        gk = W.make_grads_one(wl, k, DEV)
        for t in chosen:
            og[t].append(to_np(gk[t]))
        b = torch.empty(plan.G, device=DEV)
        B.ws_pack(plan, gk, b)
        pg.append(b)
        del gk
    ws = torch.empty(plan.workspace_bytes("lamb"), dtype=torch.uint8, device=DEV)
    B.ws_shard_update(plan, -1, pg, pw, pm, pv, hy, None, ws)
    rho_gpu = B.lamb_ratios(plan, ws).cpu().numpy().astype(np.float64)
    assert np.isfinite(rho_gpu).all() and (rho_gpu > 0).all()
    outs = {}
    for name, buf in (("w", pw), ("m", pm), ("v", pv)):
        B.ws_unpack(plan, buf, w)
        outs[name] = {t: to_np(w[t]) for t in chosen}
    worst_w = worst_mv = worst_rho = 0.0
    for t in chosen:
        rw, rm, rv = ref[t]
        rho = O.update_tensor(hs, og[t], rw, rm, rv)
        worst_rho = max(worst_rho, abs(rho_gpu[t] - rho) / rho)
        worst_w = max(worst_w, err(outs["w"][t], rw))
        worst_mv = max(worst_mv, err(outs["m"][t], rm), err(outs["v"][t], rv))
    print(f"bert_large LAMB: err w {worst_w:.2e} m/v {worst_mv:.2e} rho {worst_rho:.2e}")
    assert worst_rho <= TOL_LAMB and worst_w <= TOL_LAMB and worst_mv <= TOL_FP32


@pytest.mark.parametrize("name", ["resnet50", "transformer", "bert_large", "resnet50_lars"])
def test_benchmark_configuration_fp32_master_weights_full_size(name):
    """What bench.py times for the fp32 workloads: ws_fused_update on all shards with the weight tensors as
    the master copy (no sharded w), for BERT-large as one kernel.  Every weight tensor, m and v must equal
    the separate-kernel route bit for bit (which the tests above tie to the oracle), two steps in a row."""
    wl = W.WORKLOADS[name]()
    torch.cuda.empty_cache()
    plan = B.Plan(wl.shapes, wl.R, A)
    w, m, v = W.make_state(wl, DEV)
    has_v = wl.opt in ("adam", "lamb")
    pw = torch.empty(plan.G, device=DEV)
    pm, pv = torch.empty_like(pw), torch.empty_like(pw)
    for src, dst in ((w, pw), (m, pm), (v, pv)):
        B.ws_pack(plan, src, dst)
    fm, fv = pm.clone(), pv.clone()
    del m, v
    glists = [W.make_grads_one(wl, k, DEV) for k in range(wl.R)]
    gtab, wtab = B.TensorTable(plan, glists), B.TensorTable(plan, [w])
    ws = torch.full((max(32, plan.workspace_bytes(wl.opt)),), 0x5A, dtype=torch.uint8, device=DEV)
    ws2 = torch.full_like(ws, 0xA5)
    pg = []
    for gk in glists:
        b = torch.empty(plan.G, device=DEV)
        B.ws_pack(plan, gk, b)
        pg.append(b)
    for step in (10, 11):
        hy = B.make_hyper(wl.opt, dict(wl.hyper, step=step))
        B.ws_shard_update(plan, -1, pg, pw, pm, pv if has_v else None, hy, None, ws)
        B.ws_fused_update(plan, -1, gtab, None, fm, fv if has_v else None, hy, wtab, ws2)
    torch.cuda.synchronize()
    del pg
    assert torch.equal(fm, pm) and (not has_v or torch.equal(fv, pv))
    ref = [torch.empty_like(x) for x in w]
    B.ws_unpack(plan, pw, ref)
    for t, (a, b) in enumerate(zip(w, ref)):
        assert torch.equal(a, b), f"tensor {t}"
    if wl.opt == "lamb":
        assert torch.equal(B.lamb_ratios(plan, ws), B.lamb_ratios(plan, ws2))
        off = plan.sync_status_offset()
        assert int(ws2[off:off + 4].view(torch.int32).item()) == 0


def test_bert_large_lamb_fused_equals_unfused():
    """The benchmark's configuration for config 4: ws_fused_update (three launches) from the 16
    gradient lists.  Same arithmetic and same tiling as the packed path, so every output is
    bit-identical to ws_pack + ws_shard_update + ws_unpack (which the test above ties to the oracle)."""
    wl = W.bert_large()
    torch.cuda.empty_cache()
    plan = B.Plan(wl.shapes, wl.R, A)
    hy = B.make_hyper(wl.opt, wl.hyper)
    w, m, v = W.make_state(wl, DEV)
    pw = torch.empty(plan.G, device=DEV)
    pm, pv = torch.empty_like(pw), torch.empty_like(pw)
    for src, dst in ((w, pw), (m, pm), (v, pv)):
        B.ws_pack(plan, src, dst)
    fw, fm, fv = pw.clone(), pm.clone(), pv.clone()
    del m, v
    glists, pg = [], []
    for k in range(wl.R):
        gk = W.make_grads_one(wl, k, DEV)
        b = torch.empty(plan.G, device=DEV)
        B.ws_pack(plan, gk, b)
        pg.append(b)
        glists.append(gk)
    ws = torch.empty(plan.workspace_bytes("lamb"), dtype=torch.uint8, device=DEV)
    ws2 = torch.empty_like(ws)
    B.ws_shard_update(plan, -1, pg, pw, pm, pv, hy, None, ws)
    del pg
    ref = [torch.empty_like(x) for x in w]
    B.ws_unpack(plan, pw, ref)
    B.ws_fused_update(plan, -1, B.TensorTable(plan, glists), fw, fm, fv, hy, B.TensorTable(plan, [w]), ws2)
    assert torch.equal(B.lamb_ratios(plan, ws), B.lamb_ratios(plan, ws2))
    assert torch.equal(fw, pw) and torch.equal(fm, pm) and torch.equal(fv, pv)
    for a, b in zip(w, ref):
        assert torch.equal(a, b)


def test_resnet50_lars_full_model_every_element():
    """The ResNet-50 tensor set under LARS (the optimizer of the paper's ResNet-50 runs, Table 1), R=8,
    through the fused route the benchmark times; every element and every local rate against the oracle."""
    wl = W.resnet50_lars()
    plan = B.Plan(wl.shapes, wl.R, A)
    w, m, _ = W.make_state(wl, DEV)
    g = W.make_grads(wl, DEV)
    ow, om = [to_np(x) for x in w], [to_np(x) for x in m]
    og = [[to_np(x) for x in gk] for gk in g]
    orate = O.update_unsharded(O.make_hyper(wl.opt, wl.hyper), og, ow, om, None)
    pw = torch.empty(plan.G, device=DEV)
    pm = torch.empty_like(pw)
    B.ws_pack(plan, w, pw)
    B.ws_pack(plan, m, pm)
    ws = torch.empty(plan.workspace_bytes("lars"), dtype=torch.uint8, device=DEV)
    outs = [torch.empty_like(x) for x in w]
    B.ws_fused_update(plan, -1, B.TensorTable(plan, g), pw, pm, None, B.make_hyper(wl.opt, wl.hyper),
                      B.TensorTable(plan, [outs]), ws)
    outs_m = [torch.empty_like(x) for x in w]
    B.ws_unpack(plan, pm, outs_m)
    ew = max(err(to_np(a), b) for a, b in zip(outs, ow))
    em = max(err(to_np(a), b) for a, b in zip(outs_m, om))
    rate = B.lamb_ratios(plan, ws).cpu().numpy().astype(np.float64)
    er = float(np.max(np.abs(rate - np.array(orate)) / np.array(orate)))
    print(f"resnet50 LARS full: err w {ew:.2e} m {em:.2e} rate {er:.2e}")
    assert ew <= TOL_LAMB and em <= TOL_LAMB and er <= TOL_LAMB


def test_transformer_adafactor_whole_tensors():
    """The Transformer tensor set under Adafactor (the paper's example, with LARS, of an optimizer whose
    reduces the sharding cuts, Section 4.1), R=8, full size, through the fused route the benchmark
    times.  The oracle recomputes whole tensors (row and column sums span all shards): the embedding,
    the first and last layers with their vectors, one of each matrix shape."""
    wl = W.transformer_adafactor()
    torch.cuda.empty_cache()
    plan = B.Plan(wl.shapes, wl.R, A)
    hy = B.make_hyper(wl.opt, wl.hyper)
    hs = O.make_hyper(wl.opt, wl.hyper)
    chosen = sorted(set([0] + list(range(1, 12)) + list(range(wl.T - 14, wl.T))))
    w, _, _ = W.make_state(wl, DEV)
    f0 = W.make_factored_state(wl, plan.factored_elems, DEV)
    lay = plan.factored_layout()
    rows_, cols_, foff_, tot = O.factor_shapes(wl.shapes)
    assert tot == plan.factored_elems and [x[0] for x in lay] == foff_.tolist()
    ref_w = {t: to_np(w[t]).reshape(wl.shapes[t]) for t in chosen}
    ref_f = to_np(f0)
    pw = torch.empty(plan.G, device=DEV)
    B.ws_pack(plan, w, pw)
    g = []
    og = {t: [] for t in chosen}
    for k in range(wl.R):
        gk = W.make_grads_one(wl, k, DEV)
        for t in chosen:
            og[t].append(to_np(gk[t]))
        g.append(gk)
    ws = torch.empty(plan.workspace_bytes("adafactor"), dtype=torch.uint8, device=DEV)
    outs = [torch.empty_like(x) for x in w]
    fs = f0.clone()
    B.ws_fused_update(plan, -1, B.TensorTable(plan, g), pw, None, fs, hy, B.TensorTable(plan, [outs]), ws)
    coef = ws[:4 * plan.T].view(torch.float32).cpu().numpy().astype(np.float64)
    got_f = to_np(fs)
    worst_w = worst_f = worst_c = 0.0
    for t in chosen:
        off, nr, nc = lay[t]
        vr = ref_f[off:off + nr]
        vc = ref_f[off + nr:off + nr + nc] if nc else None
        alpha, rms_u, _ = O.adafactor_tensor(hs, og[t], ref_w[t], vr, vc)
        worst_c = max(worst_c, abs(coef[t] - alpha / max(1.0, rms_u)) / (alpha / max(1.0, rms_u)))
        worst_w = max(worst_w, err(to_np(outs[t]), ref_w[t]))
        worst_f = max(worst_f, err(got_f[off:off + nr + nc], ref_f[off:off + nr + nc]))
    print(f"transformer Adafactor: err w {worst_w:.2e} factored state {worst_f:.2e} step size {worst_c:.2e}")
    assert worst_w <= TOL_LAMB and worst_f <= TOL_LAMB and worst_c <= TOL_LAMB
    # the form the benchmark times: the fp32 weight tensors are the master copy (no sharded w); the row and
    # column sums are combined by atomic adds, so the two runs agree to rounding, not bit for bit
    master = [x.clone() for x in w]
    fs2 = f0.clone()
    ws2 = torch.empty_like(ws)
    B.ws_fused_update(plan, -1, B.TensorTable(plan, g), None, None, fs2, hy, B.TensorTable(plan, [master]), ws2)
    worst_m = max(err(to_np(master[t]), ref_w[t]) for t in chosen)
    worst_mf = max(err(to_np(fs2)[lay[t][0]:lay[t][0] + lay[t][1] + lay[t][2]],
                       ref_f[lay[t][0]:lay[t][0] + lay[t][1] + lay[t][2]]) for t in chosen)
    print(f"transformer Adafactor, weight tensors as master: err w {worst_m:.2e} factored state {worst_mf:.2e}")
    assert worst_m <= TOL_LAMB and worst_mf <= TOL_LAMB
    for t in range(wl.T):
        if wl.numels[t]:
            assert err(to_np(master[t]), to_np(outs[t]).astype(np.float64)) <= 1e-6
    # the sharded weight state and the weight tensors hold the same values
    B.ws_unpack(plan, pw, w)
    for t in chosen:
        assert torch.equal(w[t], outs[t])
