"""Helpers shared by the GPU parity tests (error metric, oracle drivers)."""
from __future__ import annotations

import numpy as np
import torch

from oracle import ws_oracle as O

TOL_FP32 = 1e-6     # momentum-SGD and Adam outputs (fp32)
TOL_LAMB = 1e-5     # LAMB weights and trust ratios
TOL_BF16 = 1e-2     # bf16 outputs


def err(x: np.ndarray, ref: np.ndarray) -> float:
    """Per-tensor error: max_i |x_i - ref_i| / max(|ref_i|, RMS(ref)).

    fp32 rounding error scales with the operands of the update, not with a
    result that cancelled to almost nothing, so each element's error is taken
    relative to its own magnitude or the tensor's RMS, whichever is larger."""
    x = np.asarray(x, dtype=np.float64).ravel()
    ref = np.asarray(ref, dtype=np.float64).ravel()
    if ref.size == 0:
        return 0.0
    assert np.isfinite(x).all() and np.isfinite(ref).all()
    rms = float(np.sqrt(np.mean(ref * ref)))
    den = np.maximum(np.abs(ref), rms)
    den[den == 0.0] = 1.0
    return float(np.max(np.abs(x - ref) / den))


def to_np(t: torch.Tensor) -> np.ndarray:
    """Device/CPU tensor -> numpy; bf16 comes back as raw uint16 bits."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16).copy()
    return t.numpy().copy()


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    return O.bf16_bits_to_f64(bits)
