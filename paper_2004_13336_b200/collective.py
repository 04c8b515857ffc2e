"""The sharded weight update across real replicas, one process per GPU (paper Section 2.2,
"Sharding with decomposed all-reduce"): every replica packs its own gradients into the
shard-major layout, a reduce-scatter leaves replica r the summed shard r, replica r updates
its 1/R of the weights and of the optimizer slots (which stay sharded between steps), and an
all-gather of the updated shards rebuilds the full weights - in bfloat16 when asked, while
the update stays fp32 (Section 4.2).  LAMB and LARS add the combination of the replicas'
partial norm sums between their two phases (Section 4.1, "Non-elementwise operators").

This module is plumbing only: the collectives are ``torch.distributed`` calls (NCCL on GPUs)
and every arithmetic step is a call into the C-ABI library through ``binding``.  The receive
buffer of the reduce-scatter is handed to the update kernel as is (``slice_mode = 1``, one
gradient copy), and the kernel writes slot r of the gathered buffer, which is the all-gather's
own input and output layout, so no extra copy sits between a collective and a kernel.

``ops`` names the module that supplies ``Plan``, ``ws_pack``, ``ws_unpack``,
``ws_shard_update``, ``ws_lamb_partial / _finalize / _apply``, ``ws_lars_partial / _finalize /
_apply``, ``lamb_partials`` and ``make_hyper``; it is the CUDA binding unless a test passes a
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
        if opt not in ("sgdm", "adam", "lamb", "lars"):
            raise ValueError("shard-by-shard updates exist for sgdm, adam, lamb and lars")
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
        if opt in ("lamb", "lars"):
            self.workspace = torch.zeros(max(16, self.plan.workspace_bytes(opt)), dtype=torch.uint8,
                                         device=self.device)

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
