"""Sharded weight update for data-parallel training on one B200 (sm_100a).

The work is done by the C-ABI CUDA library ``libws.so`` (``include/ws.h``,
sources under ``csrc/``); this package only builds it (``build.py``), loads
it and marshals arguments (``binding.py``).  The entry points carry the names
of the C functions::

    from paper_2004_13336_b200 import binding as ws
    plan = ws.Plan(shapes, R)                         # ws_plan_create + ws_plan_upload
    ws.ws_pack(plan, tensors, flat)                   # tensors -> shard-major [R][S]
    ws.ws_shard_update(plan, -1, grads, w, m, v, ws.make_hyper("adam", hyper))
    ws.ws_unpack(plan, w, tensors)
    ws.ws_fused_update(plan, -1, ws.TensorTable(plan, grad_lists), w, m, v, hyper,
                       ws.TensorTable(plan, [weight_tensors]))   # the same step in one kernel

``workloads.py`` holds the model-shaped synthetic tensor sets used by the
tests and the benchmark.  There is no CPU fallback: without the built library
every call fails at import of the binding.
"""

__all__ = ["binding", "build", "workloads"]
