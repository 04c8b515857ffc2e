"""Thin ctypes binding of libws.so: same names as the C ABI (include/ws.h),
argument marshalling only.  Every step of the path runs in the CUDA library;
there is no CPU fallback - loading fails loudly when the library is missing.

Tensors are torch tensors used purely as device memory (``data_ptr()``) and
streams come from ``torch.cuda.current_stream()``.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# WS_DEBUG_BOUNDS=1 selects the bounds-checking debug build of the library (see ws.h)
DEBUG_BOUNDS = os.environ.get("WS_DEBUG_BOUNDS", "") == "1"
LIB_PATH = os.path.join(_PKG, "libws_debug.so" if DEBUG_BOUNDS else "libws.so")

WS_OK = 0
WS_F32, WS_BF16 = 0, 1
WS_SGDM, WS_ADAM, WS_LAMB, WS_LARS = 0, 1, 2, 3
WS_ADAFACTOR = 4
OPT_CODE = {"sgdm": WS_SGDM, "adam": WS_ADAM, "lamb": WS_LAMB, "lars": WS_LARS, "adafactor": WS_ADAFACTOR}
WS_LAYOUT_PER_TENSOR, WS_LAYOUT_CONCAT = 0, 1
LAYOUT_CODE = {"per_tensor": WS_LAYOUT_PER_TENSOR, "concat": WS_LAYOUT_CONCAT}
WS_MAX_DIMS = 8


class WsError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        msg = lib().ws_status_string(status).decode()
        extra = lib().ws_last_cuda_error().decode()
        super().__init__(f"{what}: {msg}" + (f" ({extra})" if status == 6 and extra else ""))


class ws_tensor_desc(C.Structure):
    _fields_ = [("ndim", C.c_int32), ("dims", C.c_int64 * WS_MAX_DIMS), ("flags", C.c_uint32)]


class ws_segment(C.Structure):
    _fields_ = [("numel", C.c_int64), ("piece", C.c_int64), ("shard_off", C.c_int64)]


class ws_grads(C.Structure):
    _fields_ = [("ptrs", C.POINTER(C.c_void_p)), ("R", C.c_int32), ("dtype", C.c_int32),
                ("slice_mode", C.c_int32)]


class ws_state(C.Structure):
    _fields_ = [("w", C.c_void_p), ("m", C.c_void_p), ("v", C.c_void_p)]


class ws_hyper(C.Structure):
    _fields_ = [("opt", C.c_int32), ("lr", C.c_double), ("beta1", C.c_double), ("beta2", C.c_double),
                ("eps", C.c_double), ("weight_decay", C.c_double), ("momentum", C.c_double),
                ("grad_scale", C.c_double), ("step", C.c_int64), ("trust_coeff", C.c_double),
                ("eps2", C.c_double), ("clip_threshold", C.c_double), ("decay_exponent", C.c_double)]


class ws_out(C.Structure):
    _fields_ = [("gathered", C.c_void_p), ("dtype", C.c_int32)]


class ws_tensor_table(C.Structure):
    _fields_ = [("dev", C.c_void_p), ("nsets", C.c_int32), ("T", C.c_int32), ("dtype", C.c_int32),
                ("min_align", C.c_int32)]


class ws_sched_item(C.Structure):
    _fields_ = [("tensor", C.c_int32), ("shard", C.c_int32), ("pos", C.c_int64), ("tensor_off", C.c_int64),
                ("len", C.c_int32), ("nvalid", C.c_int32)]


class ws_host_io(C.Structure):
    _fields_ = [("host_grads", C.POINTER(C.c_void_p)), ("grad_dtype", C.c_int32),
                ("dev_grad_arena", C.c_void_p), ("dev_packed_grads", C.POINTER(C.c_void_p)),
                ("dev_weight_arena", C.c_void_p), ("host_weights", C.c_void_p)]


EXPORTS = [
    "ws_plan_create", "ws_plan_destroy", "ws_plan_num_tensors", "ws_plan_num_shards", "ws_plan_align",
    "ws_plan_shard_elems", "ws_plan_valid_elems", "ws_plan_num_tiles", "ws_plan_segments",
    "ws_plan_device_bytes", "ws_plan_upload", "ws_pack", "ws_unpack", "ws_workspace_bytes",
    "ws_shard_update", "ws_lamb_partial", "ws_lamb_finalize", "ws_lamb_apply", "ws_status_string",
    "ws_last_cuda_error", "ws_plan_arena_elems", "ws_plan_arena_offsets", "ws_step_host",
    "ws_static_scratch_bytes", "ws_lamb_update_static_scratch",
    "ws_tensor_table_bytes", "ws_tensor_table_upload", "ws_fused_update",
    "ws_plan_create_layout", "ws_plan_layout", "ws_pack_sets",
    "ws_plan_factored_elems", "ws_plan_factored_layout", "ws_workspace_partials",
    "ws_lars_partial", "ws_lars_finalize", "ws_lars_apply",
    "ws_adafactor_stage", "ws_workspace_adafactor_sums",
    "ws_plan_schedule_bytes", "ws_plan_upload_schedule", "ws_plan_schedule_view", "ws_plan_schedule_item",
    "ws_workspace_sync_status",
    "ws_debug_bounds_enabled", "ws_debug_bounds_read", "ws_debug_bounds_selftest",
]

_lib = None


def lib() -> C.CDLL:
    """Loads libws.so from the package directory.  Raises if it has not been
    built (``python -m paper_2004_13336_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2004_13336_b200.build` "
                          "(there is no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    vp, vpp = C.c_void_p, C.POINTER(C.c_void_p)
    L.ws_plan_create.restype = C.c_int
    L.ws_plan_create.argtypes = [C.POINTER(ws_tensor_desc), C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                 C.POINTER(vp)]
    L.ws_plan_create_layout.restype = C.c_int
    L.ws_plan_create_layout.argtypes = [C.POINTER(ws_tensor_desc), C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                        C.c_int, C.POINTER(vp)]
    L.ws_plan_layout.restype = C.c_int32
    L.ws_plan_layout.argtypes = [vp]
    L.ws_plan_destroy.restype = None
    L.ws_plan_destroy.argtypes = [vp]
    for name, rt in (("ws_plan_num_tensors", C.c_int32), ("ws_plan_num_shards", C.c_int32),
                     ("ws_plan_align", C.c_int32), ("ws_plan_shard_elems", C.c_int64),
                     ("ws_plan_valid_elems", C.c_int64), ("ws_plan_num_tiles", C.c_int64),
                     ("ws_plan_device_bytes", C.c_size_t)):
        getattr(L, name).restype = rt
        getattr(L, name).argtypes = [vp]
    L.ws_plan_segments.restype = C.c_int
    L.ws_plan_segments.argtypes = [vp, C.POINTER(C.POINTER(ws_segment)), C.POINTER(C.c_int32)]
    L.ws_plan_upload.restype = C.c_int
    L.ws_plan_upload.argtypes = [vp, vp, C.c_size_t, vp]
    L.ws_pack.restype = C.c_int
    L.ws_pack.argtypes = [vp, vpp, C.c_int, vp, vp]
    L.ws_unpack.restype = C.c_int
    L.ws_unpack.argtypes = [vp, vp, C.c_int, vpp, vp]
    L.ws_workspace_bytes.restype = C.c_size_t
    L.ws_workspace_bytes.argtypes = [vp, C.c_int]
    L.ws_shard_update.restype = C.c_int
    L.ws_shard_update.argtypes = [vp, C.c_int32, C.POINTER(ws_grads), C.POINTER(ws_state),
                                  C.POINTER(ws_hyper), C.POINTER(ws_out), vp, C.c_size_t, vp]
    L.ws_lamb_partial.restype = C.c_int
    L.ws_lamb_partial.argtypes = [vp, C.c_int32, C.POINTER(ws_grads), C.POINTER(ws_state),
                                  C.POINTER(ws_hyper), vp, C.c_size_t, vp]
    L.ws_lamb_finalize.restype = C.c_int
    L.ws_lamb_finalize.argtypes = [vp, vp, C.c_size_t, vp]
    L.ws_lamb_apply.restype = C.c_int
    L.ws_lamb_apply.argtypes = [vp, C.c_int32, C.POINTER(ws_state), C.POINTER(ws_hyper),
                                C.POINTER(ws_out), vp, C.c_size_t, vp]
    L.ws_plan_arena_elems.restype = C.c_int64
    L.ws_plan_arena_elems.argtypes = [vp]
    L.ws_lars_partial.restype = C.c_int
    L.ws_lars_partial.argtypes = [vp, C.c_int32, C.POINTER(ws_grads), C.POINTER(ws_state), C.POINTER(ws_hyper),
                                  vp, C.c_size_t, vp]
    L.ws_lars_finalize.restype = C.c_int
    L.ws_lars_finalize.argtypes = [vp, C.POINTER(ws_hyper), vp, C.c_size_t, vp]
    L.ws_lars_apply.restype = C.c_int
    L.ws_lars_apply.argtypes = [vp, C.c_int32, C.POINTER(ws_state), C.POINTER(ws_hyper), C.POINTER(ws_out),
                                vp, C.c_size_t, vp]
    L.ws_adafactor_stage.restype = C.c_int
    L.ws_adafactor_stage.argtypes = [vp, C.c_int, C.c_int32, C.POINTER(ws_grads), C.POINTER(ws_state),
                                     C.POINTER(ws_hyper), C.POINTER(ws_out), vp, C.c_size_t, vp]
    L.ws_workspace_adafactor_sums.restype = C.c_int
    L.ws_workspace_adafactor_sums.argtypes = [vp, C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
    L.ws_workspace_partials.restype = C.c_int
    L.ws_workspace_partials.argtypes = [vp, C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
    L.ws_plan_factored_elems.restype = C.c_int64
    L.ws_plan_factored_elems.argtypes = [vp]
    L.ws_plan_factored_layout.restype = C.c_int
    L.ws_plan_factored_layout.argtypes = [vp, C.POINTER(C.c_int64)]
    L.ws_plan_arena_offsets.restype = C.c_int
    L.ws_plan_arena_offsets.argtypes = [vp, C.POINTER(C.POINTER(C.c_int64)), C.POINTER(C.c_int32)]
    L.ws_step_host.restype = C.c_int
    L.ws_step_host.argtypes = [vp, C.POINTER(ws_host_io), C.POINTER(ws_state), C.POINTER(ws_hyper),
                               C.POINTER(ws_out), vp, C.c_size_t, vp]
    L.ws_static_scratch_bytes.restype = C.c_size_t
    L.ws_static_scratch_bytes.argtypes = []
    L.ws_lamb_update_static_scratch.restype = C.c_int
    L.ws_lamb_update_static_scratch.argtypes = [vp, C.POINTER(ws_grads), C.POINTER(ws_state),
                                                C.POINTER(ws_hyper), C.POINTER(ws_out), vp]
    L.ws_tensor_table_bytes.restype = C.c_size_t
    L.ws_tensor_table_bytes.argtypes = [vp, C.c_int32]
    L.ws_tensor_table_upload.restype = C.c_int
    L.ws_tensor_table_upload.argtypes = [vp, vpp, C.c_int32, C.c_int, vp, C.c_size_t, vp,
                                         C.POINTER(ws_tensor_table)]
    L.ws_pack_sets.restype = C.c_int
    L.ws_pack_sets.argtypes = [vp, C.POINTER(ws_tensor_table), vpp, vp]
    L.ws_fused_update.restype = C.c_int
    L.ws_fused_update.argtypes = [vp, C.c_int32, C.POINTER(ws_tensor_table), C.POINTER(ws_state),
                                  C.POINTER(ws_hyper), C.POINTER(ws_tensor_table), vp, C.c_size_t, vp]
    L.ws_plan_schedule_bytes.restype = C.c_size_t
    L.ws_plan_schedule_bytes.argtypes = [vp]
    L.ws_plan_upload_schedule.restype = C.c_int
    L.ws_plan_upload_schedule.argtypes = [vp, vp, C.c_size_t, vp]
    L.ws_plan_schedule_view.restype = C.c_int
    L.ws_plan_schedule_view.argtypes = [vp, C.POINTER(C.POINTER(C.c_uint32)), C.POINTER(C.c_int64)]
    L.ws_plan_schedule_item.restype = C.c_int
    L.ws_plan_schedule_item.argtypes = [vp, C.c_int64, C.POINTER(ws_sched_item)]
    L.ws_workspace_sync_status.restype = C.c_int
    L.ws_workspace_sync_status.argtypes = [vp, C.POINTER(C.c_size_t)]
    L.ws_debug_bounds_enabled.restype = C.c_int32
    L.ws_debug_bounds_enabled.argtypes = []
    L.ws_debug_bounds_read.restype = C.c_int
    L.ws_debug_bounds_read.argtypes = [C.POINTER(C.c_uint32), C.c_int32]
    L.ws_debug_bounds_selftest.restype = C.c_int
    L.ws_debug_bounds_selftest.argtypes = [vp]
    L.ws_status_string.restype = C.c_char_p
    L.ws_status_string.argtypes = [C.c_int]
    L.ws_last_cuda_error.restype = C.c_char_p
    L.ws_last_cuda_error.argtypes = []
    _lib = L
    return L


def debug_bounds_read(clear: bool = True) -> int:
    """Bits of the bounds-checking debug build's status word (synchronises the device)."""
    bits = C.c_uint32()
    _check(lib().ws_debug_bounds_read(C.byref(bits), 1 if clear else 0), "ws_debug_bounds_read")
    return bits.value


def _check(status: int, what: str):
    if status != WS_OK:
        raise WsError(status, what)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dtype_code(dt: torch.dtype) -> int:
    if dt == torch.float32:
        return WS_F32
    if dt == torch.bfloat16:
        return WS_BF16
    raise TypeError(f"unsupported dtype {dt}")


class PtrList:
    """A tensor list with its C pointer array built once, for callers that pass
    the same tensors every step (keeps the per-call host cost to one ctypes call)."""

    def __init__(self, tensors: Sequence[torch.Tensor]):
        self.tensors = list(tensors)
        self.arr = _ptr_array(self.tensors)
        self.dtype = self.tensors[0].dtype if self.tensors else torch.float32

    def __len__(self):
        return len(self.tensors)

    def __getitem__(self, i):
        return self.tensors[i]


def _ptr_array(tensors):
    if isinstance(tensors, PtrList):
        return tensors.arr
    arr = (C.c_void_p * max(1, len(tensors)))()
    for i, t in enumerate(tensors):
        arr[i] = t.data_ptr()
    return arr


def make_hyper(opt, hyper: dict) -> ws_hyper:
    code = OPT_CODE[opt] if isinstance(opt, str) else int(opt)
    return ws_hyper(code, hyper["lr"], hyper["beta1"], hyper["beta2"], hyper["eps"],
                    hyper["weight_decay"], hyper["momentum"], hyper["grad_scale"], int(hyper["step"]),
                    float(hyper.get("trust_coeff", 0.001)), float(hyper.get("eps2", 1e-3)),
                    float(hyper.get("clip_threshold", 1.0)), float(hyper.get("decay_exponent", 0.8)))


class Plan:
    """Owns a ws_plan and the device buffer that holds its tables."""

    def __init__(self, shapes: Sequence[Sequence[int]], R: int, align_elems: int = 32, tile_elems: int = 0,
                 device: Optional[torch.device] = None, upload: bool = True, layout: str = "per_tensor",
                 one_launch: bool = True):
        """``one_launch``: also upload the plan's one-launch schedule, so that the all-shard LAMB and LARS
        updates run as one kernel (with ``False`` they run as three launches)."""
        T = len(shapes)
        descs = (ws_tensor_desc * max(1, T))()
        for i, s in enumerate(shapes):
            s = tuple(int(x) for x in s)
            if len(s) > WS_MAX_DIMS:
                s = (int(torch.Size(s).numel()),)
            descs[i].ndim = len(s)
            for j, d in enumerate(s):
                descs[i].dims[j] = d
        self._h = C.c_void_p()
        self.layout = layout
        _check(lib().ws_plan_create_layout(descs, T, R, align_elems, tile_elems, LAYOUT_CODE[layout],
                                           C.byref(self._h)), "ws_plan_create_layout")
        L = lib()
        self.T, self.R, self.A = L.ws_plan_num_tensors(self._h), L.ws_plan_num_shards(self._h), L.ws_plan_align(self._h)
        self.S, self.N = L.ws_plan_shard_elems(self._h), L.ws_plan_valid_elems(self._h)
        self.G = self.R * self.S
        self.ntiles = L.ws_plan_num_tiles(self._h)
        self.dev_buf = None
        self.sched_buf = None
        if upload:
            self.upload(device)
            if one_launch:
                self.upload_schedule(device)

    @property
    def handle(self):
        return self._h

    def segments(self) -> List[ws_segment]:
        segs, T = C.POINTER(ws_segment)(), C.c_int32()
        _check(lib().ws_plan_segments(self._h, C.byref(segs), C.byref(T)), "ws_plan_segments")
        return [segs[i] for i in range(T.value)]

    def upload(self, device=None):
        nbytes = lib().ws_plan_device_bytes(self._h)
        self.dev_buf = torch.empty(nbytes, dtype=torch.uint8, device=device or "cuda")
        _check(lib().ws_plan_upload(self._h, self.dev_buf.data_ptr(), nbytes, _stream()), "ws_plan_upload")

    def upload_schedule(self, device=None):
        nbytes = lib().ws_plan_schedule_bytes(self._h)
        if nbytes == 0:          # the plan has no one-launch schedule
            return
        self.sched_buf = torch.empty(nbytes, dtype=torch.uint8, device=device or "cuda")
        _check(lib().ws_plan_upload_schedule(self._h, self.sched_buf.data_ptr(), nbytes, _stream()),
               "ws_plan_upload_schedule")

    def schedule(self):
        """(order, items): the one-launch execution order as a list of (item, phase) and the items as
        ws_sched_item records.  Host only."""
        order, n = C.POINTER(C.c_uint32)(), C.c_int64()
        _check(lib().ws_plan_schedule_view(self._h, C.byref(order), C.byref(n)), "ws_plan_schedule_view")
        import numpy as np
        arr = np.ctypeslib.as_array(order, shape=(n.value,)).copy()
        items = []
        for i in range(n.value // 2):
            it = ws_sched_item()
            _check(lib().ws_plan_schedule_item(self._h, i, C.byref(it)), "ws_plan_schedule_item")
            items.append(it)
        return [(int(e) >> 1, int(e) & 1) for e in arr], items

    def sync_status_offset(self) -> int:
        off = C.c_size_t()
        _check(lib().ws_workspace_sync_status(self._h, C.byref(off)), "ws_workspace_sync_status")
        return off.value

    @property
    def arena_elems(self) -> int:
        return lib().ws_plan_arena_elems(self._h)

    def arena_offsets(self) -> List[int]:
        offs, T = C.POINTER(C.c_int64)(), C.c_int32()
        _check(lib().ws_plan_arena_offsets(self._h, C.byref(offs), C.byref(T)), "ws_plan_arena_offsets")
        return [offs[i] for i in range(T.value)]

    def arena_views(self, arena: torch.Tensor, numels: Sequence[int]) -> List[torch.Tensor]:
        """Per-tensor views of a tensor arena (host or device)."""
        return [arena[o:o + n] for o, n in zip(self.arena_offsets(), numels)]

    @property
    def factored_elems(self) -> int:
        """Floats of Adafactor's factored second-moment state for all tensors."""
        return lib().ws_plan_factored_elems(self._h)

    def factored_layout(self):
        """Per tensor (offset, rows, cols) of its factored state; cols == 0: unfactored, rows = numel."""
        buf = (C.c_int64 * (3 * max(1, self.T)))()
        _check(lib().ws_plan_factored_layout(self._h, buf), "ws_plan_factored_layout")
        return [(buf[3 * t], buf[3 * t + 1], buf[3 * t + 2]) for t in range(self.T)]

    def workspace_bytes(self, opt) -> int:
        code = OPT_CODE[opt] if isinstance(opt, str) else int(opt)
        return lib().ws_workspace_bytes(self._h, code)

    def __del__(self):
        try:
            if self._h:
                lib().ws_plan_destroy(self._h)
                self._h = None
        except Exception:
            pass


def ws_pack(plan: Plan, tensors: Sequence[torch.Tensor], flat: torch.Tensor):
    dt = _dtype_code(flat.dtype)
    _check(lib().ws_pack(plan.handle, _ptr_array(tensors), dt, flat.data_ptr(), _stream()), "ws_pack")


def ws_unpack(plan: Plan, flat: torch.Tensor, tensors: Sequence[torch.Tensor]):
    dt = _dtype_code(flat.dtype)
    _check(lib().ws_unpack(plan.handle, flat.data_ptr(), dt, _ptr_array(tensors), _stream()), "ws_unpack")


def _grads(gbufs: Sequence[torch.Tensor], slice_mode: int):
    arr = _ptr_array(gbufs)
    g = ws_grads(C.cast(arr, C.POINTER(C.c_void_p)), len(gbufs), _dtype_code(gbufs[0].dtype), slice_mode)
    g._keep = arr
    return g


def _state(w, m, v):
    return ws_state(w.data_ptr() if w is not None else None, m.data_ptr() if m is not None else None,
                    v.data_ptr() if v is not None else None)


def _out(gathered):
    if gathered is None:
        return None
    return ws_out(gathered.data_ptr(), _dtype_code(gathered.dtype))


def ws_shard_update(plan: Plan, r: int, gbufs: Sequence[torch.Tensor], w, m, v, hyper: ws_hyper,
                    gathered: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                    slice_mode: int = 0):
    g, s, o = _grads(gbufs, slice_mode), _state(w, m, v), _out(gathered)
    _check(lib().ws_shard_update(plan.handle, r, C.byref(g), C.byref(s), C.byref(hyper),
                                 C.byref(o) if o is not None else None,
                                 workspace.data_ptr() if workspace is not None else None,
                                 workspace.numel() * workspace.element_size() if workspace is not None else 0,
                                 _stream()), "ws_shard_update")


def ws_lamb_partial(plan: Plan, r: int, gbufs, w, m, v, hyper: ws_hyper, workspace: torch.Tensor,
                    slice_mode: int = 0):
    g, s = _grads(gbufs, slice_mode), _state(w, m, v)
    _check(lib().ws_lamb_partial(plan.handle, r, C.byref(g), C.byref(s), C.byref(hyper), workspace.data_ptr(),
                                 workspace.numel() * workspace.element_size(), _stream()), "ws_lamb_partial")


def ws_lamb_finalize(plan: Plan, workspace: torch.Tensor):
    _check(lib().ws_lamb_finalize(plan.handle, workspace.data_ptr(),
                                  workspace.numel() * workspace.element_size(), _stream()), "ws_lamb_finalize")


def ws_lamb_apply(plan: Plan, r: int, w, m, v, hyper: ws_hyper, workspace: torch.Tensor,
                  gathered: Optional[torch.Tensor] = None):
    s, o = _state(w, m, v), _out(gathered)
    _check(lib().ws_lamb_apply(plan.handle, r, C.byref(s), C.byref(hyper),
                               C.byref(o) if o is not None else None, workspace.data_ptr(),
                               workspace.numel() * workspace.element_size(), _stream()), "ws_lamb_apply")


def ws_lars_partial(plan: Plan, r: int, gbufs, w, m, hyper: ws_hyper, workspace: torch.Tensor, slice_mode: int = 0):
    g, s = _grads(gbufs, slice_mode), _state(w, m, None)
    _check(lib().ws_lars_partial(plan.handle, r, C.byref(g), C.byref(s), C.byref(hyper), workspace.data_ptr(),
                                 workspace.numel() * workspace.element_size(), _stream()), "ws_lars_partial")


def ws_lars_finalize(plan: Plan, hyper: ws_hyper, workspace: torch.Tensor):
    _check(lib().ws_lars_finalize(plan.handle, C.byref(hyper), workspace.data_ptr(),
                                  workspace.numel() * workspace.element_size(), _stream()), "ws_lars_finalize")


def ws_lars_apply(plan: Plan, r: int, w, m, hyper: ws_hyper, workspace: torch.Tensor,
                  gathered: Optional[torch.Tensor] = None):
    s, o = _state(w, m, None), _out(gathered)
    _check(lib().ws_lars_apply(plan.handle, r, C.byref(s), C.byref(hyper), C.byref(o) if o is not None else None,
                               workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream()),
           "ws_lars_apply")


AF_BEGIN, AF_SUMS, AF_MOMENTS, AF_SUMSQ, AF_CLIP, AF_APPLY = range(6)


def ws_adafactor_stage(plan: Plan, stage: int, r: int, hyper: ws_hyper, workspace: torch.Tensor, gbufs=None,
                       w=None, fstate=None, gathered: Optional[torch.Tensor] = None, slice_mode: int = 0):
    """One stage of Adafactor (AF_BEGIN ... AF_APPLY) for shard r, or all shards with r = -1."""
    g = _grads(gbufs, slice_mode) if gbufs is not None else None
    s = ws_state(w.data_ptr() if w is not None else None, None, fstate.data_ptr() if fstate is not None else None)
    o = _out(gathered)
    _check(lib().ws_adafactor_stage(plan.handle, stage, r, C.byref(g) if g is not None else None, C.byref(s),
                                    C.byref(hyper), C.byref(o) if o is not None else None, workspace.data_ptr(),
                                    workspace.numel() * workspace.element_size(), _stream()), "ws_adafactor_stage")


def adafactor_sums(plan: Plan, workspace: torch.Tensor) -> torch.Tensor:
    """Float view of this step's row / column sums inside an Adafactor workspace (the all-reduce operand)."""
    off, nb = C.c_size_t(), C.c_size_t()
    _check(lib().ws_workspace_adafactor_sums(plan.handle, C.byref(off), C.byref(nb)), "ws_workspace_adafactor_sums")
    return workspace[off.value: off.value + nb.value].view(torch.float32)


def lamb_partials(plan: Plan, workspace: torch.Tensor) -> torch.Tensor:
    """The [R][tiles * 2] float view of the per-tile partial sums inside a LAMB workspace."""
    off, row = C.c_size_t(), C.c_size_t()
    _check(lib().ws_workspace_partials(plan.handle, C.byref(off), C.byref(row)), "ws_workspace_partials")
    return workspace[off.value: off.value + plan.R * row.value].view(torch.float32).view(plan.R, row.value // 4)


def lamb_ratios(plan: Plan, workspace: torch.Tensor) -> torch.Tensor:
    """The trust ratios rho[T] that ws_lamb_finalize left at the start of the workspace."""
    return workspace[: 4 * plan.T].view(torch.float32)


def ws_step_host(plan: Plan, host_grads: Sequence[torch.Tensor], dev_grad_arena: torch.Tensor,
                 dev_packed_grads: Sequence[torch.Tensor], w, m, v, hyper: ws_hyper,
                 dev_weight_arena: torch.Tensor, host_weights: torch.Tensor,
                 gathered: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None):
    """Host gradient arenas in, host weight arena out (pinned memory for overlap-free async copies)."""
    hg, dp = _ptr_array(host_grads), _ptr_array(dev_packed_grads)
    io = ws_host_io(C.cast(hg, C.POINTER(C.c_void_p)), _dtype_code(host_grads[0].dtype),
                    dev_grad_arena.data_ptr(), C.cast(dp, C.POINTER(C.c_void_p)),
                    dev_weight_arena.data_ptr(), host_weights.data_ptr())
    s, o = _state(w, m, v), _out(gathered)
    _check(lib().ws_step_host(plan.handle, C.byref(io), C.byref(s), C.byref(hyper),
                              C.byref(o) if o is not None else None,
                              workspace.data_ptr() if workspace is not None else None,
                              workspace.numel() * workspace.element_size() if workspace is not None else 0,
                              _stream()), "ws_step_host")


def ws_lamb_update_static_scratch(plan: Plan, gbufs, w, m, v, hyper: ws_hyper,
                                  gathered: Optional[torch.Tensor] = None):
    """LAMB update of all shards for callers that cannot provide a workspace: the scratch
    is a fixed array inside the library (see ws.h for its size limit and sharing rules)."""
    g, s, o = _grads(gbufs, 0), _state(w, m, v), _out(gathered)
    _check(lib().ws_lamb_update_static_scratch(plan.handle, C.byref(g), C.byref(s), C.byref(hyper),
                                               C.byref(o) if o is not None else None, _stream()),
           "ws_lamb_update_static_scratch")


class TensorTable:
    """Device-resident table of tensor pointers for ws_fused_update: `sets` is a list of
    tensor lists (R gradient lists, or one weight list).  Keeps the device buffer alive."""

    def __init__(self, plan: Plan, sets: Sequence[Sequence[torch.Tensor]], device=None):
        nsets = len(sets)
        flat = [t for s in sets for t in s]
        assert len(flat) == nsets * plan.T
        self.sets = [list(s) for s in sets]
        nbytes = lib().ws_tensor_table_bytes(plan.handle, nsets)
        if device is None:      # the table itself always lives on the GPU
            device = flat[0].device if flat[0].is_cuda else plan.dev_buf.device
        self.dev_buf = torch.empty(nbytes, dtype=torch.uint8, device=device)
        self.c = ws_tensor_table()
        _check(lib().ws_tensor_table_upload(plan.handle, _ptr_array(flat), nsets, _dtype_code(flat[0].dtype),
                                            self.dev_buf.data_ptr(), nbytes, _stream(), C.byref(self.c)),
               "ws_tensor_table_upload")

    @classmethod
    def from_pointers(cls, plan: Plan, ptr_sets: Sequence[Sequence[int]], dtype: torch.dtype, device):
        """The same table from raw device addresses (sets of T integers) - for tensors that live in
        another process's memory mapped into this one (CUDA IPC, symmetric memory).  The caller keeps
        the mappings alive."""
        self = cls.__new__(cls)
        nsets = len(ptr_sets)
        flat = [int(p) for s in ptr_sets for p in s]
        assert len(flat) == nsets * plan.T
        self.sets = None
        nbytes = lib().ws_tensor_table_bytes(plan.handle, nsets)
        self.dev_buf = torch.empty(nbytes, dtype=torch.uint8, device=device)
        self.c = ws_tensor_table()
        arr = (C.c_void_p * max(1, len(flat)))(*flat)
        _check(lib().ws_tensor_table_upload(plan.handle, arr, nsets, _dtype_code(dtype), self.dev_buf.data_ptr(),
                                            nbytes, _stream(), C.byref(self.c)), "ws_tensor_table_upload")
        return self


def ws_fused_update(plan: Plan, r: int, grads: TensorTable, w, m, v, hyper: ws_hyper, weights: TensorTable,
                    workspace: Optional[torch.Tensor] = None):
    s = _state(w, m, v)
    _check(lib().ws_fused_update(plan.handle, r, C.byref(grads.c), C.byref(s), C.byref(hyper), C.byref(weights.c),
                                 workspace.data_ptr() if workspace is not None else None,
                                 workspace.numel() * workspace.element_size() if workspace is not None else 0,
                                 _stream()), "ws_fused_update")


def ws_pack_sets(plan: Plan, table: TensorTable, flats):
    """All sets of a tensor table packed in one launch (set k -> flats[k])."""
    _check(lib().ws_pack_sets(plan.handle, C.byref(table.c), _ptr_array(flats), _stream()), "ws_pack_sets")
