"""Image-quality measures for focused point targets (test infrastructure).

Impulse-response width (IRW, the -3 dB width of the main lobe, in bins) and
peak sidelobe ratio (PSLR, dB) along one image axis, as the paper reports them
for its reference image (Section "End to End", "Processing and validation").
These are measurements of an image, not steps of the method.
"""
from __future__ import annotations

import numpy as np


def _upsample(cut: np.ndarray, factor: int) -> np.ndarray:
    """Band-limited interpolation of a 1-D complex cut by spectrum zero padding."""
    n = cut.size
    spec = np.fft.fft(cut)
    pad = np.zeros(n * factor, dtype=np.complex128)
    h = n // 2
    pad[:h] = spec[:h]
    pad[-(n - h):] = spec[h:]
    return np.fft.ifft(pad) * factor


def cut_through(image: np.ndarray, cell, axis: int, half: int = 64) -> np.ndarray:
    a, r = cell
    if axis == 0:
        return image[a - half:a + half, r].copy()
    return image[a, r - half:r + half].copy()


def irw_pslr(cut: np.ndarray, factor: int = 32):
    """(-3 dB width in original bins, PSLR in dB, peak offset in bins from the
    cut centre) of a 1-D complex cut whose peak is near the centre."""
    up = np.abs(_upsample(np.asarray(cut, dtype=np.complex128), factor))
    pk = int(np.argmax(up))
    peak = up[pk]
    thr = peak / np.sqrt(2.0)

    def cross(direction):
        i = pk
        while 0 < i < up.size - 1 and up[i] >= thr:
            i += direction
        j = i - direction                      # last sample above the threshold
        frac = (up[j] - thr) / (up[j] - up[i]) if up[j] != up[i] else 0.0
        return j + direction * frac

    width = (cross(+1) - cross(-1)) / factor

    def first_null(direction):
        i = pk
        while 0 < i + direction < up.size - 1 and up[i + direction] <= up[i]:
            i += direction
        return i

    lo, hi = first_null(-1), first_null(+1)
    side = max(up[:lo].max() if lo > 0 else 0.0, up[hi + 1:].max() if hi + 1 < up.size else 0.0)
    pslr = 20.0 * np.log10(side / peak) if side > 0 else -np.inf
    offset = pk / factor - cut.size // 2
    return width, pslr, offset


def peak_cell(image: np.ndarray, cell, half: int = 8):
    """argmax of |image| in a +-half window around `cell` (ties: lowest index)."""
    a, r = cell
    a0, r0 = max(a - half, 0), max(r - half, 0)
    win = np.abs(image[a0:a + half + 1, r0:r + half + 1])
    i = int(np.argmax(win))
    return (a0 + i // win.shape[1], r0 + i % win.shape[1])
