"""World-size-2 and -3 CPU runs (gloo) of the multi-replica choreography of Section 2.2 -
pack, reduce-scatter, update of the own shard from the receive buffer, all-gather, unpack -
with the oracle standing in for the CUDA kernels.  Checks that every rank ends with the
weights of the plain unsharded update and that the slots stay sharded and gather back."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

SHAPES = [(1,), (7,), (3, 3, 4, 8), (64, 33), (1031,), (5, 1, 9)]


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _inputs(world):
    from paper_2004_13336_b200 import workloads as W
    wl = W.Workload("t", list(SHAPES), R=world, opt="adam", hyper={}, grad_std=1e-2, seed=17)
    w, m, v = W.make_state(wl, "cpu")
    g = W.make_grads(wl, "cpu")
    return wl, w, m, v, g


def _hyper_for(opt, world):
    h = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0, momentum=0.9, grad_scale=1.0 / world, step=3)
    if opt == "sgdm":
        h.update(lr=0.1, weight_decay=5e-5)
    if opt == "lamb":
        h.update(eps=1e-6, weight_decay=0.01)
    if opt == "lars":
        h.update(lr=2.0, weight_decay=5e-5, trust_coeff=0.02)
    if opt == "adafactor":
        h.update(lr=1e-2, beta1=0.0, beta2=0.0, eps=1e-30, eps2=1e-3, clip_threshold=1.0, decay_exponent=0.8)
    return h


def _fstate0(n):
    gen = torch.Generator().manual_seed(5)
    return torch.rand(n, generator=gen) * 1e-3 + 1e-6


def _worker(rank, world, port, opt, out_bf16, out):
    from oracle import ws_oracle as O
    from paper_2004_13336_b200.collective import ShardedUpdate
    from tests import _oracle_ops
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl, w, m, v, g = _inputs(world)
    hyper = _hyper_for(opt, world)
    su = ShardedUpdate(SHAPES, opt, hyper, out_dtype=torch.bfloat16 if out_bf16 else torch.float32,
                       device="cpu", ops=_oracle_ops)
    su.load_state(w, m, v)
    if opt == "adafactor":
        su.fstate.copy_(_fstate0(su.plan.factored_elems))
    outs = [torch.zeros(n, dtype=su.gathered.dtype) for n in wl.numels]
    su.step(g[rank], outs)                       # this rank's own gradients only
    m_full = [torch.zeros(n) for n in wl.numels]
    su.gather_slot(su.m, m_full)
    if opt == "adafactor":
        m_full = [su.fstate.numpy().copy()]      # the (replicated) factored state instead of a momentum
    ratios = _oracle_ops.lamb_ratios(su.plan, su.workspace).numpy().copy() if opt in ("lamb", "lars") else None
    out[rank] = ([o.view(torch.int16).numpy().copy() if out_bf16 else o.numpy().copy() for o in outs],
                 [np.asarray(x).copy() for x in m_full], ratios)
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
@pytest.mark.parametrize("opt,out_bf16", [("adam", False), ("sgdm", True)])
def test_every_rank_ends_with_the_unsharded_result(world, opt, out_bf16):
    from oracle import ws_oracle as O
    port = _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, opt, out_bf16, out), nprocs=world, join=True)
        res = dict(out)
    # expected: the plain update of whole tensors from the all-reduced gradient (summed in fp32 in
    # rank order, as the collective does for world 2; for world 3 the association may differ by an ulp)
    wl, w, m, v, g = _inputs(world)
    hyper = _hyper_for(opt, world)
    hs = O.make_hyper(opt, hyper)
    for t in range(wl.T):
        gs = g[0][t].clone()
        for k in range(1, world):
            gs += g[k][t]
        ew, em = w[t].numpy().copy(), m[t].numpy().copy()
        ev = v[t].numpy().copy() if opt == "adam" else None
        O.update_tensor(hs, [gs.numpy()], ew, em, ev)
        for rank in range(world):
            got_w, got_m = res[rank][0][t], res[rank][1][t]
            if out_bf16:
                exp = O.f32_to_bf16_bits(ew)
                assert (np.abs(got_w.view(np.uint16).astype(np.int64) - exp.astype(np.int64)) <= (0 if world == 2 else 1)).all()
            elif world == 2:
                np.testing.assert_array_equal(got_w, ew)
                np.testing.assert_array_equal(got_m, em)
            else:
                np.testing.assert_allclose(got_w, ew, rtol=0, atol=1e-7)
                np.testing.assert_allclose(got_m, em, rtol=1e-5, atol=1e-9)
    for rank in range(1, world):                 # all ranks hold identical full weights
        for a, b in zip(res[0][0], res[rank][0]):
            np.testing.assert_array_equal(a, b)


@pytest.mark.parametrize("world", [2, 3])
@pytest.mark.parametrize("opt,out_bf16", [("lamb", False), ("lars", True)])
def test_norm_based_optimizers_exchange_their_partial_sums(world, opt, out_bf16):
    """LAMB and LARS on CPU ranks (Section 4.1: every replica reduces what its shard holds, then the
    replicas combine their partial reduce results): phase 1 on the rank's own shard, all-gather of the
    partial rows, the same combination on every rank, phase 2, all-gather of the weights.  Every rank
    must end with the unsharded oracle result and all ranks with identical ratios."""
    from oracle import ws_oracle as O
    port = _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, opt, out_bf16, out), nprocs=world, join=True)
        res = dict(out)
    wl, w, m, v, g = _inputs(world)
    hs = O.make_hyper(opt, _hyper_for(opt, world))
    for rank in range(1, world):                 # identical weights, slots and ratios everywhere
        for a, b in zip(res[0][0], res[rank][0]):
            np.testing.assert_array_equal(a, b)
        np.testing.assert_array_equal(res[0][2], res[rank][2])
    for t in range(wl.T):
        gs = g[0][t].clone()
        for k in range(1, world):                # the collective's fp32 sum in rank order
            gs += g[k][t]
        ew, em = w[t].numpy().copy(), m[t].numpy().copy()
        ev = v[t].numpy().copy() if opt == "lamb" else None
        rho = O.update_tensor(hs, [gs.numpy()], ew, em, ev)
        # (the sharded route sums a tensor's norm shard by shard: the ratio agrees to double rounding, the
        # weights to one fp32 ulp; with three ranks the collective may also associate the sum differently)
        assert abs(res[0][2][t] / rho - 1.0) < 1e-6
        got_w, got_m = res[0][0][t], res[0][1][t]
        if out_bf16:
            exp = O.f32_to_bf16_bits(ew)
            assert (np.abs(got_w.view(np.uint16).astype(np.int64) - exp.astype(np.int64)) <= 1).all()
        else:
            np.testing.assert_allclose(got_w, ew, rtol=0, atol=2e-7)
        np.testing.assert_allclose(got_m, em, rtol=1e-5, atol=1e-9)


@pytest.mark.parametrize("world", [2, 3])
def test_adafactor_combines_row_and_column_sums_across_ranks(world):
    """Adafactor on CPU ranks (Section 4.1: a reduce whose collapsed dimension the sharding cuts - every
    replica reduces what its shard holds, then the replicas combine their results with an all-reduce):
    the stages of one replica around the all-reduce of the row / column sums and the exchange of the
    scalar partial sums.  Every rank must end with the unsharded oracle result and the same factored state."""
    from oracle import ws_oracle as O
    port = _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, "adafactor", False, out), nprocs=world, join=True)
        res = dict(out)
    wl, w, m, v, g = _inputs(world)
    hs = O.make_hyper("adafactor", _hyper_for("adafactor", world))
    for rank in range(1, world):
        for a, b in zip(res[0][0], res[rank][0]):
            np.testing.assert_array_equal(a, b)
        np.testing.assert_array_equal(res[0][1][0], res[rank][1][0])
    rows, cols, foff, F = O.factor_shapes(SHAPES)
    f = _fstate0(F).numpy().copy()
    for t in range(wl.T):
        gs = g[0][t].clone()
        for k in range(1, world):
            gs += g[k][t]
        ew = w[t].numpy().copy().reshape(SHAPES[t])
        vr = f[foff[t]:foff[t] + rows[t]]
        vc = f[foff[t] + rows[t]:foff[t] + rows[t] + cols[t]] if cols[t] else None
        O.adafactor_tensor(hs, [gs.numpy()], ew, vr, vc)
        np.testing.assert_allclose(res[0][0][t], ew.ravel(), rtol=0, atol=2e-7)
    np.testing.assert_allclose(res[0][1][0], f, rtol=2e-7, atol=0)
