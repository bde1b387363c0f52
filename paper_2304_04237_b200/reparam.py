"""Re-parameterisation utility of the deformed shifting module (Sec. 4.3, Fig. 4): the training-time
form has two parallel depthwise paths -- the fixed one-hot shift kernels of Eq. 11 and randomly
initialised learned kernels -- whose outputs add; at inference they merge into ONE depthwise
convolution whose kernel is the sum of the two.  The library's forward takes that merged kernel.

Host-side helpers (numpy); nothing here runs on the hot path.
"""
from __future__ import annotations

import numpy as np


def shift_kernels(channels: int, ksize: int) -> np.ndarray:
    """The fixed shift kernels (Eq. 11) as the library lays weights out: float32 [C][k*k slot][k*k tap],
    1 where tap == slot."""
    k2 = ksize * ksize
    w = np.zeros((channels, k2, k2), dtype=np.float32)
    idx = np.arange(k2)
    w[:, idx, idx] = 1.0
    return w


def merge_two_path(learned: np.ndarray, ksize: int) -> np.ndarray:
    """Merged kernel = fixed shift + learned (Sec. 4.3).  `learned`: [C][k*k][k*k] in the library's
    layout, or a PyTorch depthwise weight [C*k*k, 1, k, k] with groups = C (output channel c*k*k + s)."""
    k2 = ksize * ksize
    w = np.asarray(learned, dtype=np.float32)
    if w.ndim == 4:
        assert w.shape[1:] == (1, ksize, ksize) and w.shape[0] % k2 == 0
        w = w.reshape(w.shape[0] // k2, k2, k2)
    assert w.ndim == 3 and w.shape[1:] == (k2, k2)
    return (shift_kernels(w.shape[0], ksize) + w).astype(np.float32)


def split_merged(merged: np.ndarray, ksize: int) -> np.ndarray:
    """The learned part of a merged kernel (merged - fixed shift): what training would go on from."""
    w = np.asarray(merged, dtype=np.float32)
    return (w - shift_kernels(w.shape[0], ksize)).astype(np.float32)
