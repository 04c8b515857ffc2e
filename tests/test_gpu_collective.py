"""The multi-replica route of Section 2.2 (pack, NCCL reduce-scatter, update of the own shard
from the receive buffer, NCCL all-gather, unpack) on the GPU.  A run has one GPU, so the
process group has one rank: the collectives are real NCCL calls on a world of one and the
kernels run exactly as rank r of R would run them (single shard, slice_mode 1, LAMB in its
three per-shard phases with the partial sums exchanged).  Ranks > 1 are covered on CPU
(tests/test_collective_cpu.py)."""
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist

from oracle import ws_oracle as O
from paper_2004_13336_b200 import workloads as W
from paper_2004_13336_b200.collective import ShardedUpdate
from tests._util import TOL_BF16, TOL_FP32, TOL_LAMB, bf16_to_f64, err, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda"
SHAPES = [(1,), (7,), (3, 3, 16, 32), (64, 128), (1031,), (5, 1, 9), (4099, 3), (300, 301)]


@pytest.fixture(scope="module")
def world_of_one():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1)
    yield
    dist.destroy_process_group()


@pytest.mark.parametrize("opt,out_dtype,gdtype", [("sgdm", torch.float32, torch.float32),
                                                  ("adam", torch.bfloat16, torch.bfloat16),
                                                  ("lamb", torch.float32, torch.float32),
                                                  ("lamb", torch.bfloat16, torch.float32),
                                                  ("lars", torch.float32, torch.float32)])
def test_one_rank_group_matches_the_oracle(world_of_one, opt, out_dtype, gdtype):
    wl = W.Workload("t", list(SHAPES), R=1, opt=opt, hyper={}, grad_dtype=gdtype, grad_std=1e-2, seed=23)
    w, m, v = W.make_state(wl, DEV)
    g = W.make_grads(wl, DEV)[0]
    hyper = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-6, weight_decay=0.01 if opt != "adam" else 0.0,
                 momentum=0.9, grad_scale=1.0, step=4)
    if opt == "lars":
        hyper.update(lr=10.0, weight_decay=5e-5, trust_coeff=0.001)
    su = ShardedUpdate(SHAPES, opt, hyper, out_dtype=out_dtype, grad_dtype=gdtype, device=DEV)
    su.load_state(w, m, v)
    outs = [torch.zeros(n, dtype=out_dtype, device=DEV) for n in wl.numels]
    for step in (4, 5):                       # two steps: the sharded slots carry over
        hyper["step"] = step
        su.step(g, outs, step=step)
    torch.cuda.synchronize()
    ow, om, ov = [to_np(x) for x in w], [to_np(x) for x in m], [to_np(x) for x in v]
    og = [to_np(x) for x in g]
    for step in (4, 5):
        hyper["step"] = step
        O.update_unsharded(O.make_hyper(opt, hyper), [og], ow, om, ov if opt in ("adam", "lamb") else None)
    tol = TOL_LAMB if opt in ("lamb", "lars") else 2 * TOL_FP32
    for t, (a, b) in enumerate(zip(outs, ow)):
        if out_dtype == torch.bfloat16:
            assert err(bf16_to_f64(to_np(a)), b) <= TOL_BF16, t
        else:
            assert err(to_np(a), b) <= tol, t
    m_full = [torch.zeros(n, device=DEV) for n in wl.numels]
    su.gather_slot(su.m, m_full)
    for t, (a, b) in enumerate(zip(m_full, om)):
        assert err(to_np(a), b) <= tol, t


@pytest.mark.parametrize("opt,out_dtype,gdtype", [("sgdm", torch.float32, torch.float32),
                                                  ("adam", torch.bfloat16, torch.bfloat16)])
def test_one_kernel_route_over_symmetric_memory(world_of_one, opt, out_dtype, gdtype):
    """The peer-mapped route on a world of one: the arenas are symmetric memory, the tables hold
    the addresses the rendezvous returned, one kernel does the whole step."""
    from paper_2004_13336_b200.collective import PeerShardedUpdate
    wl = W.Workload("t", list(SHAPES), R=1, opt=opt, hyper={}, grad_dtype=gdtype, grad_std=1e-2, seed=29)
    w, m, v = W.make_state(wl, DEV)
    g = W.make_grads(wl, DEV)[0]
    hyper = dict(lr=1e-2, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=5e-5 if opt == "sgdm" else 0.0,
                 momentum=0.9, grad_scale=1.0, step=2)
    try:
        pu = PeerShardedUpdate(SHAPES, opt, hyper, out_dtype=out_dtype, grad_dtype=gdtype, device=DEV)
    except (RuntimeError, NotImplementedError) as e:      # no symmetric-memory support in this environment
        pytest.skip(f"symmetric memory unavailable: {str(e)[:120]}")
    pu.load_state(w, m, v)
    for dst, src in zip(pu.grads, g):
        dst.copy_(src)
    pu.step()
    torch.cuda.synchronize()
    ow, om, ov = [to_np(x) for x in w], [to_np(x) for x in m], [to_np(x) for x in v]
    O.update_unsharded(O.make_hyper(opt, hyper), [[to_np(x) for x in g]], ow, om, ov if opt == "adam" else None)
    for t, (a, b) in enumerate(zip(pu.weights, ow)):
        if out_dtype == torch.bfloat16:
            assert err(bf16_to_f64(to_np(a)), b) <= TOL_BF16, t
        else:
            assert err(to_np(a), b) <= TOL_FP32, t


def test_adafactor_on_a_one_rank_group(world_of_one):
    """Adafactor on the NCCL route: per-shard stages with the all-reduce of the row / column sums and the
    exchange of the per-tile sums between them (real NCCL calls, one rank)."""
    shapes = SHAPES + [(24, 2048)]
    wl = W.Workload("t", list(shapes), R=1, opt="adafactor", hyper={}, grad_std=1e-2, seed=37)
    w, m, v = W.make_state(wl, DEV)
    g = W.make_grads(wl, DEV)[0]
    hyper = dict(lr=1e-2, beta1=0.0, beta2=0.0, eps=1e-30, weight_decay=0.0, momentum=0.0, grad_scale=1.0, step=3,
                 eps2=1e-3, clip_threshold=1.0, decay_exponent=0.8)
    su = ShardedUpdate(shapes, "adafactor", hyper, device=DEV)
    su.load_state(w, m, v)
    f0 = W.make_factored_state(wl, su.plan.factored_elems, DEV)
    su.fstate.copy_(f0)
    outs = [torch.zeros(n, device=DEV) for n in wl.numels]
    su.step(g, outs)
    torch.cuda.synchronize()
    hs = O.make_hyper("adafactor", hyper)
    of = to_np(f0)
    for t, (off, rows, cols) in enumerate(su.plan.factored_layout()):
        ref = to_np(w[t]).reshape(shapes[t])
        O.adafactor_tensor(hs, [to_np(g[t])], ref, of[off:off + rows], of[off + rows:off + rows + cols] if cols else None)
        assert err(to_np(outs[t]), ref) <= TOL_LAMB, t
        assert err(to_np(su.fstate)[off:off + rows + cols], of[off:off + rows + cols]) <= TOL_LAMB, t
