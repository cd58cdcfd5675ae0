"""Host-side helpers for the rotation tables that `hf_set_rope` takes (the library itself only consumes angles).

`relative_temporal_indices` is Eq. 8: the temporal index of a chunk's frames counts up with the stream until the
largest index T_0 the pretrained model has seen, then stays there.  `angle_tables` turns per-token (t, y, x)
positions into cos / sin tables [T, d/2] with the usual rotary frequencies, the d/2 pairs split over the three axes.
"""
from __future__ import annotations

import numpy as np


def relative_temporal_indices(last_frame: int, t0: int, chunk_frames: int = 3):
    """Temporal indices of the `chunk_frames` frames of the chunk whose last frame is the stream's (1-based) frame
    `last_frame`: [last - c + 1, ..., last] while last <= t0, else [t0 - c + 1, ..., t0]  (Eq. 8 for c = 3)."""
    top = last_frame if last_frame <= t0 else t0
    return [top - chunk_frames + 1 + i for i in range(chunk_frames)]


def angle_tables(positions: np.ndarray, pairs_per_axis, base: float = 10000.0):
    """positions: int array [T, A] (one coordinate per axis); pairs_per_axis: A counts summing to d/2.
    Pair j of axis a rotates by position[a] * base ** (-j / pairs_per_axis[a]).  Returns float32 (cos, sin) [T, d/2]."""
    positions = np.asarray(positions, dtype=np.float64)
    cols = []
    for a, n in enumerate(pairs_per_axis):
        freq = base ** (-np.arange(n, dtype=np.float64) / n)
        cols.append(positions[:, a:a + 1] * freq[None, :])
    th = np.concatenate(cols, axis=1)
    return np.cos(th).astype(np.float32), np.sin(th).astype(np.float32)


def chunk_positions(last_frame: int, t0: int, chunk_frames: int, height: int, width: int) -> np.ndarray:
    """(t, y, x) of every token of a chunk in frame-major, row-major order, temporal index per Eq. 8."""
    ts = relative_temporal_indices(last_frame, t0, chunk_frames)
    t, y, x = np.meshgrid(np.asarray(ts), np.arange(height), np.arange(width), indexing="ij")
    return np.stack([t.ravel(), y.ravel(), x.ravel()], axis=1)
