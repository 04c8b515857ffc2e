"""Stand-in for the CUDA binding on CPU ranks: the same call names as
``paper_2004_13336_b200.binding`` (the subset ``collective.ShardedUpdate`` uses), computed by the
oracle on numpy views of CPU tensors.  Test infrastructure only: it lets world-size-2 gloo tests
run the reduce-scatter / update / all-gather choreography without a GPU."""
import numpy as np
import torch

from oracle import ws_oracle as O


class Plan:
    def __init__(self, shapes, R, align_elems=32, tile_elems=0, device=None, upload=True, layout="per_tensor"):
        self.numels = [int(np.prod(s)) for s in shapes]
        self.o = O.Plan(self.numels, R, align_elems)
        self.S, self.G, self.T, self.R = self.o.S, self.o.G, self.o.T, R

    def workspace_bytes(self, opt):
        return 0


def make_hyper(opt, hyper):
    return O.make_hyper(opt, hyper)


def _np(t):
    """numpy view sharing memory with the CPU tensor; bf16 as raw uint16 bits."""
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def ws_pack(plan, tensors, flat):
    flat.copy_(torch.from_numpy(O.pack(plan.o, [_np(t).ravel() for t in tensors])))


def ws_unpack(plan, flat, outs):
    for dst, src in zip(outs, O.unpack(plan.o, _np(flat))):
        if dst.dtype == torch.bfloat16:
            dst.copy_(torch.from_numpy(src.view(np.int16)).view(torch.bfloat16).view_as(dst))
        else:
            dst.copy_(torch.from_numpy(src).view_as(dst))


def ws_shard_update(plan, r, gbufs, w, m, v, hyper, gathered=None, workspace=None, slice_mode=0):
    """Shard r from its reduce-scatter receive buffer (slice_mode 1, one gradient copy): the
    optimizers here are elementwise, so each tensor's valid piece is updated as a tensor of its own."""
    assert slice_mode == 1 and len(gbufs) == 1 and 0 <= r < plan.R
    g, wn, mn = _np(gbufs[0]), _np(w), _np(m)
    vn = _np(v) if v is not None else None
    for t in range(plan.T):
        p, off, n = int(plan.o.piece[t]), int(plan.o.off[t]), int(plan.o.numel[t])
        nv = min(max(n - r * p, 0), p)
        sl = slice(off, off + nv)
        if nv:
            wt, mt = wn[sl].copy(), mn[sl].copy()
            vt = vn[sl].copy() if vn is not None else None
            O.update_tensor(hyper, [np.ascontiguousarray(g[sl])], wt, mt, vt)
            wn[sl], mn[sl] = wt, mt
            if vn is not None:
                vn[sl] = vt
        for a in (wn, mn, vn):
            if a is not None:
                a[off + nv:off + p] = 0.0
    if gathered is not None:
        slot = gathered[r * plan.S:(r + 1) * plan.S]
        if gathered.dtype == torch.bfloat16:
            slot.copy_(torch.from_numpy(O.f32_to_bf16_bits(wn).view(np.int16)).view(torch.bfloat16))
        else:
            slot.copy_(w)
