"""The sharded weight update across real replicas, one process per GPU (paper Section 2.2,
"Sharding with decomposed all-reduce"): every replica packs its own gradients into the
shard-major layout, a reduce-scatter leaves replica r the summed shard r, replica r updates
its 1/R of the weights and of the optimizer slots (which stay sharded between steps), and an
all-gather of the updated shards rebuilds the full weights - in bfloat16 when asked, while
the update stays fp32 (Section 4.2).  LAMB and LARS add the combination of the replicas'
partial norm sums between their two phases, Adafactor the all-reduce of its row / column sums
(Section 4.1, "Non-elementwise operators").

This module is plumbing only: the collectives are ``torch.distributed`` calls (NCCL on GPUs)
and every arithmetic step is a call into the C-ABI library through ``binding``.  The receive
buffer of the reduce-scatter is handed to the update kernel as is (``slice_mode = 1``, one
gradient copy), and the kernel writes slot r of the gathered buffer, which is the all-gather's
own input and output layout, so no extra copy sits between a collective and a kernel.

``ops`` names the module that supplies ``Plan``, ``ws_pack``, ``ws_unpack``,
``ws_shard_update``, ``ws_lamb_partial / _finalize / _apply``, ``ws_lars_partial / _finalize /
_apply``, ``ws_adafactor_stage``, ``lamb_partials``, ``adafactor_sums`` and ``make_hyper``; it is the CUDA binding unless a test passes a
stand-in to run the choreography on CPU ranks.
"""
from __future__ import annotations

from typing import Dict, Optional, Sequence

import torch
import torch.distributed as dist


class ShardedUpdate:
    """Replica ``rank`` of ``world`` replicas.  Holds shard ``rank`` of w, m, v (fp32, S elements
    each) and the full gathered weights ([R][S] of ``out_dtype``)."""

    def __init__(self, shapes: Sequence[Sequence[int]], opt: str, hyper: Dict[str, float],
                 out_dtype: torch.dtype = torch.float32, grad_dtype: torch.dtype = torch.float32,
                 align_elems: int = 32, device=None, group=None, ops=None):
        if ops is None:
            from . import binding as ops      # fails loudly without the built CUDA library
        if opt not in ("sgdm", "adam", "lamb", "lars", "adafactor"):
            raise ValueError(f"unknown optimizer {opt}")
        self.ops, self.opt, self.hyper_dict, self.group = ops, opt, dict(hyper), group
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)
        self.device = torch.device(device) if device is not None else torch.device("cuda", torch.cuda.current_device())
        self.plan = ops.Plan(shapes, self.world, align_elems, device=self.device)
        S, G = self.plan.S, self.plan.G
        z = dict(dtype=torch.float32, device=self.device)
        self.w, self.m, self.v = torch.zeros(S, **z), torch.zeros(S, **z), torch.zeros(S, **z)
        self.packed = torch.empty(G, dtype=grad_dtype, device=self.device)    # reduce-scatter input
        self.recv = torch.empty(S, dtype=grad_dtype, device=self.device)      # ... and output
        self.gathered = torch.zeros(G, dtype=out_dtype, device=self.device)   # all-gather buffer
        self.workspace = None
        if opt in ("lamb", "lars", "adafactor"):
            self.workspace = torch.zeros(max(16, self.plan.workspace_bytes(opt)), dtype=torch.uint8,
                                         device=self.device)
        self.fstate = None                                                    # Adafactor: replicated, small
        if opt == "adafactor":
            self.fstate = torch.zeros(self.plan.factored_elems, **z)

    # -- sharding program (Section 4.2): every replica starts from the same full state -----
    def load_state(self, w: Sequence[torch.Tensor], m: Sequence[torch.Tensor], v: Sequence[torch.Tensor]):
        S, r = self.plan.S, self.rank
        full = torch.empty(self.plan.G, dtype=torch.float32, device=self.device)
        for src, dst in ((w, self.w), (m, self.m), (v, self.v)):
            self.ops.ws_pack(self.plan, src, full)
            dst.copy_(full[r * S:(r + 1) * S])

    # -- unsharding program: the full slot tensors, for a checkpoint ------------------------
    def gather_slot(self, shard: torch.Tensor, out: Sequence[torch.Tensor]):
        full = torch.empty(self.plan.G, dtype=torch.float32, device=self.device)
        dist.all_gather_into_tensor(full, shard, group=self.group)
        self.ops.ws_unpack(self.plan, full, out)

    def step(self, grads: Sequence[torch.Tensor], weights_out: Sequence[torch.Tensor], step: Optional[int] = None):
        """One training step's weight update.  ``grads``: this replica's local gradients, one tensor
        per model tensor.  ``weights_out``: the model's weight tensors (``out_dtype``), overwritten
        with the updated full weights."""
        ops, plan, r, S = self.ops, self.plan, self.rank, self.plan.S
        if step is not None:
            self.hyper_dict["step"] = step
        hy = ops.make_hyper(self.opt, self.hyper_dict)
        ops.ws_pack(plan, grads, self.packed)                                   # formatting (Section 5.1)
        dist.reduce_scatter_tensor(self.recv, self.packed, op=dist.ReduceOp.SUM, group=self.group)
        if self.opt == "lamb":
            ops.ws_lamb_partial(plan, r, [self.recv], self.w, self.m, self.v, hy, self.workspace, slice_mode=1)
            rows = ops.lamb_partials(plan, self.workspace)                      # [R][tiles * 2]
            dist.all_gather_into_tensor(rows.view(-1), rows[r], group=self.group)
            ops.ws_lamb_finalize(plan, self.workspace)                          # same sums, same order, every rank
            ops.ws_lamb_apply(plan, r, self.w, self.m, self.v, hy, self.workspace, self.gathered)
        elif self.opt == "adafactor":
            # Section 4.1, reduces over a sharded dimension: every replica reduces what its shard holds,
            # then the results are combined with an all-reduce (here also the per-tile scalar sums)
            st, ws = ops.ws_adafactor_stage, self.workspace
            rows = ops.lamb_partials(plan, ws)
            st(plan, ops.AF_BEGIN, -1, hy, ws)
            st(plan, ops.AF_SUMS, r, hy, ws, gbufs=[self.recv], w=self.w, slice_mode=1)
            dist.all_reduce(ops.adafactor_sums(plan, ws), group=self.group)
            dist.all_gather_into_tensor(rows.view(-1), rows[r], group=self.group)
            st(plan, ops.AF_MOMENTS, -1, hy, ws, fstate=self.fstate)
            st(plan, ops.AF_SUMSQ, r, hy, ws)
            dist.all_gather_into_tensor(rows.view(-1), rows[r], group=self.group)
            st(plan, ops.AF_CLIP, -1, hy, ws)
            st(plan, ops.AF_APPLY, r, hy, ws, w=self.w, gathered=self.gathered)
        elif self.opt == "lars":
            ops.ws_lars_partial(plan, r, [self.recv], self.w, self.m, hy, self.workspace, slice_mode=1)
            rows = ops.lamb_partials(plan, self.workspace)
            dist.all_gather_into_tensor(rows.view(-1), rows[r], group=self.group)
            ops.ws_lars_finalize(plan, hy, self.workspace)
            ops.ws_lars_apply(plan, r, self.w, self.m, hy, self.workspace, self.gathered)
        else:
            ops.ws_shard_update(plan, r, [self.recv], self.w, self.m, self.v if self.opt == "adam" else None,
                                hy, self.gathered, None, slice_mode=1)
        dist.all_gather_into_tensor(self.gathered, self.gathered[r * S:(r + 1) * S], group=self.group)
        ops.ws_unpack(plan, self.gathered, weights_out)                         # reverse formatting


class PeerShardedUpdate:
    """The same step as ONE kernel per replica over peer-mapped tensors (Section 5.1: the formatting
    fused into the reduce-scatter and into the all-gather).  Every replica keeps its gradient tensors
    and its weight tensors in a symmetric-memory arena that all replicas of the NVLink domain map;
    replica r's ``ws_fused_update(plan, r, ...)`` reads its slice of every replica's gradients with
    plain peer loads, updates shard r, and stores the new weights into every replica's weight tensors
    with plain peer stores.  No packed buffer, no receive buffer, no gathered buffer exist.  Two
    stream-ordered NCCL barriers bracket the kernel: every replica's gradients are complete before any
    kernel reads them, and every replica's shard has landed before the weights are used.

    ``grads`` / ``weights``: this replica's tensors (views into the arenas) - the backward pass leaves
    its gradients in ``grads``, the forward pass reads ``weights``.  Elementwise optimizers only.
    Not run on more than one GPU so far."""

    def __init__(self, shapes: Sequence[Sequence[int]], opt: str, hyper: Dict[str, float],
                 out_dtype: torch.dtype = torch.float32, grad_dtype: torch.dtype = torch.float32,
                 align_elems: int = 32, device=None, group=None):
        import torch.distributed._symmetric_memory as symm
        from . import binding as B
        if opt not in ("sgdm", "adam"):
            raise ValueError("one-kernel replica updates exist for sgdm and adam")
        self.B, self.opt, self.hyper_dict = B, opt, dict(hyper)
        self.group = group if group is not None else dist.group.WORLD
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)
        self.device = torch.device(device) if device is not None else torch.device("cuda", torch.cuda.current_device())
        self.plan = B.Plan(shapes, self.world, align_elems, device=self.device)
        numels = [int(torch.Size(s).numel()) for s in shapes]
        n_el, offs = self.plan.arena_elems, self.plan.arena_offsets()
        self.grad_arena = symm.empty(n_el, dtype=grad_dtype, device=self.device)
        self.weight_arena = symm.empty(n_el, dtype=out_dtype, device=self.device)
        hg = symm.rendezvous(self.grad_arena, self.group)
        hw = symm.rendezvous(self.weight_arena, self.group)
        self._handles = (hg, hw)          # keep the peer mappings alive
        eg, ew = self.grad_arena.element_size(), self.weight_arena.element_size()
        self.gtab = B.TensorTable.from_pointers(
            self.plan, [[int(hg.buffer_ptrs[k]) + o * eg for o in offs] for k in range(self.world)], grad_dtype, self.device)
        self.wtab = B.TensorTable.from_pointers(
            self.plan, [[int(hw.buffer_ptrs[k]) + o * ew for o in offs] for k in range(self.world)], out_dtype, self.device)
        self.grads = self.plan.arena_views(self.grad_arena, numels)
        self.weights = self.plan.arena_views(self.weight_arena, numels)
        z = dict(dtype=torch.float32, device=self.device)
        S = self.plan.S
        self.w, self.m, self.v = torch.zeros(S, **z), torch.zeros(S, **z), torch.zeros(S, **z)
        self._token = torch.zeros(1, **z)

    def load_state(self, w: Sequence[torch.Tensor], m: Sequence[torch.Tensor], v: Sequence[torch.Tensor]):
        S, r = self.plan.S, self.rank
        full = torch.empty(self.plan.G, dtype=torch.float32, device=self.device)
        for src, dst in ((w, self.w), (m, self.m), (v, self.v)):
            self.B.ws_pack(self.plan, src, full)
            dst.copy_(full[r * S:(r + 1) * S])
        for dst, src in zip(self.weights, w):
            dst.copy_(src.reshape(-1))

    def step(self, step: Optional[int] = None):
        if step is not None:
            self.hyper_dict["step"] = step
        hy = self.B.make_hyper(self.opt, self.hyper_dict)
        dist.all_reduce(self._token, group=self.group)     # all replicas' gradients are in place
        self.B.ws_fused_update(self.plan, self.rank, self.gtab, self.w, self.m,
                               self.v if self.opt == "adam" else None, hy, self.wtab, None)
        dist.all_reduce(self._token, group=self.group)     # all shards have been stored into these weights
