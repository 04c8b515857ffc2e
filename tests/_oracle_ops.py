"""Stand-in for the CUDA binding on CPU ranks: the same call names as
``paper_2004_13336_b200.binding`` (the subset ``collective.ShardedUpdate`` uses), computed by the
oracle on numpy views of CPU tensors.  Test infrastructure only: it lets world-size-2 gloo tests
run the reduce-scatter / update / all-gather choreography without a GPU."""
import numpy as np
import torch

from oracle import ws_oracle as O


class Plan:
    def __init__(self, shapes, R, align_elems=32, tile_elems=0, device=None, upload=True, layout="per_tensor"):
        self.shapes = [tuple(int(d) for d in s) for s in shapes]
        self.factored_elems = int(O.factor_shapes(self.shapes)[3])
        self.numels = [int(np.prod(s)) for s in shapes]
        self.o = O.Plan(self.numels, R, align_elems)
        self.S, self.G, self.T, self.R = self.o.S, self.o.G, self.o.T, R

        self._u = {}          # shard -> what phase 1 keeps for phase 2 (the kernels recompute or store it)

    def workspace_bytes(self, opt):
        """Stand-in workspace for the norm-based optimizers: double rho[T] | double partials[R][T][2]."""
        if opt == "adafactor":               # ... followed by double acc[F], this step's row / column sums
            return 8 * (self.T + self.R * 2 * self.T + self.factored_elems)
        return 8 * (self.T + self.R * 2 * self.T) if opt in ("lamb", "lars") else 0


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


# ---------------------------------------------------------------- LAMB / LARS on CPU ranks ---
# Phase 1 for the rank's own shard, the exchange of the partial rows, the combination (every rank,
# same order) and phase 2: the oracle's per-replica phase functions behind the binding's call names.
def lamb_partials(plan, workspace):
    """The [R][T * 2] view of the per-shard partial sums (doubles here) inside the stand-in workspace."""
    return workspace[8 * plan.T: 8 * (plan.T + plan.R * 2 * plan.T)].view(torch.float64).view(plan.R, 2 * plan.T)


def lamb_ratios(plan, workspace):
    return workspace[:8 * plan.T].view(torch.float64)


def _partial(plan, r, gbufs, w, m, v, hyper, workspace, slice_mode):
    assert slice_mode == 1 and len(gbufs) == 1 and 0 <= r < plan.R
    part, u = O.norm_shard_partial(hyper, plan.o, r, _np(gbufs[0]), _np(w), _np(m) if m is not None else None,
                                   _np(v) if v is not None else None)
    plan._u[r] = u
    lamb_partials(plan, workspace)[r].copy_(torch.from_numpy(part.reshape(-1)))


def ws_lamb_partial(plan, r, gbufs, w, m, v, hyper, workspace, slice_mode=0):
    _partial(plan, r, gbufs, w, m, v, hyper, workspace, slice_mode)


def ws_lars_partial(plan, r, gbufs, w, m, hyper, workspace, slice_mode=0):
    _partial(plan, r, gbufs, w, None, None, hyper, workspace, slice_mode)


def _finalize(plan, hyper, workspace):
    rows = lamb_partials(plan, workspace).numpy().reshape(plan.R, plan.T, 2)
    tot = np.zeros((plan.T, 2))
    for r in range(plan.R):                   # ascending r on every rank: identical ratios everywhere
        tot += rows[r]
    lamb_ratios(plan, workspace).copy_(torch.tensor([O.norm_ratio(hyper, a, b) for a, b in tot], dtype=torch.float64))


def ws_lamb_finalize(plan, workspace, hyper=None):
    _finalize(plan, O.make_hyper("lamb", dict(lr=0, beta1=0, beta2=0, eps=0, weight_decay=0, momentum=0,
                                                 grad_scale=1, step=1)), workspace)


def ws_lars_finalize(plan, hyper, workspace):
    _finalize(plan, hyper, workspace)


def _apply(plan, r, w, m, hyper, workspace, gathered):
    out_dt = None
    if gathered is not None:
        out_dt = O.BF16 if gathered.dtype == torch.bfloat16 else O.F32
    slot = O.norm_shard_apply(hyper, plan.o, r, lamb_ratios(plan, workspace).numpy(), plan._u.pop(r), _np(w),
                              _np(m) if m is not None else None, out_dt)
    if gathered is not None:
        dst = gathered[r * plan.S:(r + 1) * plan.S]
        if gathered.dtype == torch.bfloat16:
            dst.copy_(torch.from_numpy(slot.view(np.int16)).view(torch.bfloat16))
        else:
            dst.copy_(torch.from_numpy(slot))


def ws_lamb_apply(plan, r, w, m, v, hyper, workspace, gathered=None):
    _apply(plan, r, w, None, hyper, workspace, gathered)


def ws_lars_apply(plan, r, w, m, hyper, workspace, gathered=None):
    _apply(plan, r, w, m, hyper, workspace, gathered)


# ------------------------------------------------------------------ Adafactor on CPU ranks ---
AF_BEGIN, AF_SUMS, AF_MOMENTS, AF_SUMSQ, AF_CLIP, AF_APPLY = range(6)


def adafactor_sums(plan, workspace):
    """This step's row / column sums (the all-reduce operand between AF_SUMS and AF_MOMENTS)."""
    return workspace[8 * (plan.T + plan.R * 2 * plan.T):].view(torch.float64)


def ws_adafactor_stage(plan, stage, r, hyper, workspace, gbufs=None, w=None, fstate=None, gathered=None, slice_mode=0):
    """One stage for the rank's own shard (or a replicated stage, r = -1): the oracle's per-replica stage
    functions behind the binding's call."""
    rows = lamb_partials(plan, workspace)
    if stage == AF_BEGIN:
        adafactor_sums(plan, workspace).zero_()
    elif stage == AF_SUMS:
        assert slice_mode == 1 and len(gbufs) == 1 and 0 <= r < plan.R
        rep = O.AdafactorReplica(hyper, plan.o, plan.shapes, r)
        rep.sums(_np(gbufs[0]), _np(w))
        adafactor_sums(plan, workspace).copy_(torch.from_numpy(rep.acc))
        rows[r][0::2] = torch.from_numpy(rep.pw)
        plan._af = rep
    elif stage == AF_MOMENTS:
        plan._af.moments(adafactor_sums(plan, workspace).numpy(), _np(fstate))
    elif stage == AF_SUMSQ:
        plan._af.sumsq()
        rows[r][1::2] = torch.from_numpy(plan._af.pu)
    elif stage == AF_CLIP:
        sw, su = np.zeros(plan.T), np.zeros(plan.T)
        for k in range(plan.R):                       # ascending shard order on every rank
            sw += rows[k][0::2].numpy()
            su += rows[k][1::2].numpy()
        plan._af_step = plan._af.step_sizes(sw, su)
    elif stage == AF_APPLY:
        out_dt = None if gathered is None else (O.BF16 if gathered.dtype == torch.bfloat16 else O.F32)
        slot = plan._af.apply(plan._af_step[0], plan._af_step[1], _np(w), out_dt)
        if gathered is not None:
            dst = gathered[r * plan.S:(r + 1) * plan.S]
            if gathered.dtype == torch.bfloat16:
                dst.copy_(torch.from_numpy(slot.view(np.int16)).view(torch.bfloat16))
            else:
                dst.copy_(torch.from_numpy(slot))
    else:
        raise ValueError(stage)
