"""Delayed-scaling state for one tensor class.  Test infrastructure only.

The paper describes delayed scaling as deriving scaling factors from moving
amax histories, read by one invocation and updated for the next (Sec. 2.1), and
requires the update to happen exactly once per forward and once per input-grad
action (Eqs. 3-5, Invariant 1).  The formula itself is fixed by the build's
target: scale = fp8_max / max(history) / 2^margin.  Readings taken here:

  * all arithmetic in IEEE binary32, round to nearest: one divide, one multiply
    by 2^-margin (exact unless it underflows), one divide for the inverse;
  * the newest amax enters the window before the scale for the NEXT action is
    derived, so the scale used at an action never depends on that action's data;
  * a window whose maximum is zero or not finite leaves scale and inverse alone;
  * a scale that overflows to +Inf is clamped to the largest finite binary32;
  * the history is a ring of H entries written at position (count mod H); what
    is compared between implementations is the logical window, newest first.
"""
from __future__ import annotations

import numpy as np

from .fp8 import FP8Format

_FLT_MAX = np.float32(np.finfo(np.float32).max)


class ScaleState:
    def __init__(self, fmt: FP8Format, history_len: int, margin: int):
        self.fmt = fmt
        self.H = int(history_len)
        self.margin = int(margin)
        self.hist = np.zeros(self.H, dtype=np.float32)
        self.count = 0  # number of commits so far
        self.scale = np.float32(1.0)
        self.scale_inv = np.float32(1.0)

    def commit(self, amax: np.float32) -> None:
        self.hist[self.count % self.H] = np.float32(amax)
        self.count += 1
        m = np.float32(self.hist.max())  # NaN propagates through numpy's max
        if np.isfinite(m) and m > 0:
            with np.errstate(over="ignore"):
                s = np.float32(self.fmt.max_finite) / m
                s = np.float32(s * np.float32(2.0 ** (-self.margin)))
            if np.isinf(s):
                s = _FLT_MAX
            self.scale = np.float32(s)
            self.scale_inv = np.float32(np.float32(1.0) / self.scale)

    def window(self) -> np.ndarray:
        """History as a logical window, newest first, length H (zeros where never written)."""
        idx = [(self.count - 1 - j) % self.H for j in range(self.H)]
        return self.hist[idx].copy()

    def snapshot(self) -> dict:
        return {
            "window": self.window(),
            "scale": np.float32(self.scale),
            "scale_inv": np.float32(self.scale_inv),
            "count": self.count,
        }


def amax_bf16(x_f32: np.ndarray) -> np.float32:
    """Largest magnitude of a tensor, as binary32 (exact and order-free)."""
    x = np.asarray(x_f32, dtype=np.float32)
    if x.size == 0:
        return np.float32(0.0)
    return np.float32(np.max(np.abs(x)))
