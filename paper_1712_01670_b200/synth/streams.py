"""Seeded synthetic video streams.

Pure input generation: this module draws pixels and nothing else.  It holds no
block matching, region or convolution arithmetic, so both the CPU oracle's
tests and the CUDA path's tests can feed on it without sharing any of the
method itself.

Every stream object offers random access: ``frame(i)`` renders frame ``i``
without rendering its predecessors.  All per-frame parameters (pan, patch
positions, velocities) are drawn once, in the constructor, from
``numpy.random.Generator(PCG64(seed))``; pixel noise inside a frame comes from
a generator seeded by (seed, frame index), so a frame's content depends on
nothing but the seed and its index.

The streams stand in for the UCF101 / driving videos the paper measured on
(Section 7.1); those are not available, so the shapes follow the paper's
227x227 matcher workload and five stated workload recipes.
"""
from __future__ import annotations

import numpy as np

BASE_SEED = 171201670


def _rng(*key: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([int(k) for k in key]))


# --------------------------------------------------------------------------
# value-noise canvas
# --------------------------------------------------------------------------
def value_noise_canvas(size: int, seed: int) -> np.ndarray:
    """Toroidal value-noise texture, ``size x size x 3`` uint8.

    Four octaves with lattice periods 64/32/16/8 px and amplitudes 1, 1/2, 1/4,
    1/8; each octave is a random lattice (independent per channel) interpolated
    bilinearly with wrap-around, so the canvas tiles seamlessly.
    """
    assert size % 64 == 0
    rng = _rng(seed, 0xCA7A5)
    acc = np.zeros((size, size, 3), dtype=np.float32)
    total = 0.0
    for period, amp in ((64, 1.0), (32, 0.5), (16, 0.25), (8, 0.125)):
        n = size // period
        lat = rng.random((n, n, 3)).astype(np.float32)
        pos = np.arange(size, dtype=np.float64) / period
        i0 = np.floor(pos).astype(np.int64) % n
        i1 = (i0 + 1) % n
        f = (pos - np.floor(pos)).astype(np.float32)
        # separable bilinear interpolation: along x on the lattice rows, then along y
        rows = lat[:, i0] * (1 - f)[None, :, None] + lat[:, i1] * f[None, :, None]
        acc += np.float32(amp) * (rows[i0] * (1 - f)[:, None, None] + rows[i1] * f[:, None, None])
        total += amp
    lo, hi = float(acc.min()), float(acc.max())
    acc -= np.float32(lo)
    acc *= np.float32(255.0 / (hi - lo))
    np.rint(acc, out=acc)
    return np.clip(acc, 0, 255).astype(np.uint8)


def _crop_wrap(canvas: np.ndarray, oy: int, ox: int, h: int, w: int) -> np.ndarray:
    size = canvas.shape[0]
    ys = (np.arange(h) + oy) % size
    xs = (np.arange(w) + ox) % size
    return canvas[ys[:, None], xs[None, :]]


def _pan_path(rng: np.random.Generator, n_frames: int, max_speed: int) -> np.ndarray:
    """Accumulated integer pan offsets, shape (n_frames, 2) as (oy, ox)."""
    speed = rng.integers(0, max_speed + 1, size=n_frames)
    angle = rng.random(n_frames) * 2.0 * np.pi
    step = np.stack([np.rint(speed * np.sin(angle)), np.rint(speed * np.cos(angle))], 1).astype(np.int64)
    step[0] = 0
    return np.cumsum(step, axis=0)


# --------------------------------------------------------------------------
# workload 1: one shifted pair
# --------------------------------------------------------------------------
class ShiftedPair:
    """Two 64x64 frames: frame 1 is frame 0 with content moved +3 px in x and
    -2 px in y (edge replicate), one 16x16 patch redrawn, plus N(0, 2^2) noise."""

    width = 64
    height = 64
    n_frames = 2
    n_streams = 1

    def __init__(self, seed: int = BASE_SEED + 1):
        rng = _rng(seed)
        h, w = self.height, self.width
        self.f0 = rng.integers(0, 256, size=(h, w, 3), dtype=np.uint8)
        ys = np.clip(np.arange(h) + 2, 0, h - 1)
        xs = np.clip(np.arange(w) - 3, 0, w - 1)
        f1 = self.f0[ys[:, None], xs[None, :]].astype(np.float64)
        self.patch_y = int(rng.integers(0, h - 16 + 1))
        self.patch_x = int(rng.integers(0, w - 16 + 1))
        f1[self.patch_y:self.patch_y + 16, self.patch_x:self.patch_x + 16] = rng.integers(
            0, 256, size=(16, 16, 3))
        f1 += rng.normal(0.0, 2.0, size=f1.shape)
        self.f1 = np.clip(np.rint(f1), 0, 255).astype(np.uint8)

    def frame(self, i: int, stream: int = 0) -> np.ndarray:
        return (self.f0, self.f1)[i]


# --------------------------------------------------------------------------
# workloads 2-5: panned canvas with disturbances
# --------------------------------------------------------------------------
class PannedStream:
    """Value-noise canvas seen through a panning window, plus a disturbance.

    disturbance:
      "rects"    three 32x32 solid-colour rectangles with their own velocities
      "patches"  ``n_patches`` fresh uniform-noise squares of ``patch`` px per frame
      "window"   one moving window of fresh noise covering ``window_frac`` of the
                 area, and a per-frame zoom in [1-zoom, 1+zoom] about the centre
    """

    def __init__(self, width: int, height: int, n_frames: int, seed: int, *,
                 canvas: int = 512, max_pan: int = 3, disturbance: str = "rects",
                 patch: int = 24, n_patches: int = 0, window_frac: float = 0.0,
                 zoom: float = 0.0, canvas_array: np.ndarray | None = None):
        self.width, self.height, self.n_frames, self.seed = width, height, n_frames, seed
        self.disturbance, self.patch, self.n_patches = disturbance, patch, n_patches
        self.zoom = zoom
        self.canvas = canvas_array if canvas_array is not None else value_noise_canvas(canvas, seed)
        rng = _rng(seed, 0x9A77)
        self.pan = _pan_path(rng, n_frames, max_pan)
        if disturbance == "rects":
            self.rect_pos0 = np.stack([rng.integers(0, height - 32, size=3),
                                       rng.integers(0, width - 32, size=3)], 1)
            self.rect_vel = rng.integers(-4, 5, size=(3, 2))
            self.rect_col = rng.integers(0, 256, size=(3, 3), dtype=np.uint8)
        elif disturbance == "patches":
            self.patch_yx = np.stack(
                [rng.integers(0, height - patch + 1, size=(n_frames, n_patches)),
                 rng.integers(0, width - patch + 1, size=(n_frames, n_patches))], 2)
        elif disturbance == "window":
            side_h = int(round(height * np.sqrt(window_frac)))
            side_w = int(round(width * np.sqrt(window_frac)))
            self.win_hw = (side_h, side_w)
            self.win_pos0 = np.array([rng.integers(0, height - side_h), rng.integers(0, width - side_w)])
            self.win_vel = rng.integers(-5, 6, size=2)
            self.zooms = 1.0 + (rng.random(n_frames) * 2.0 - 1.0) * zoom
        else:
            raise ValueError(disturbance)

    @staticmethod
    def _bounce(p0: int, v: int, i: int, span: int) -> int:
        """Position of a point bouncing inside [0, span]."""
        if span <= 0:
            return 0
        q = (p0 + v * i) % (2 * span)
        return int(q if q <= span else 2 * span - q)

    def _zoomed(self, img: np.ndarray, z: float) -> np.ndarray:
        h, w = img.shape[:2]
        cy, cx = (h - 1) / 2.0, (w - 1) / 2.0
        sy = np.clip((np.arange(h) - cy) / z + cy, 0, h - 1)
        sx = np.clip((np.arange(w) - cx) / z + cx, 0, w - 1)
        y0 = np.floor(sy).astype(np.int64); y1 = np.minimum(y0 + 1, h - 1); fy = (sy - y0)[:, None, None]
        x0 = np.floor(sx).astype(np.int64); x1 = np.minimum(x0 + 1, w - 1); fx = (sx - x0)[None, :, None]
        f = img.astype(np.float64)
        top = f[y0][:, x0] * (1 - fx) + f[y0][:, x1] * fx
        bot = f[y1][:, x0] * (1 - fx) + f[y1][:, x1] * fx
        return np.clip(np.rint(top * (1 - fy) + bot * fy), 0, 255).astype(np.uint8)

    def frame(self, i: int) -> np.ndarray:
        h, w = self.height, self.width
        oy, ox = self.pan[i]
        out = np.ascontiguousarray(_crop_wrap(self.canvas, int(oy), int(ox), h, w))
        noise = _rng(self.seed, 0xF2A3E, i)
        if self.disturbance == "rects":
            for r in range(3):
                y = self._bounce(int(self.rect_pos0[r, 0]), int(self.rect_vel[r, 0]), i, h - 32)
                x = self._bounce(int(self.rect_pos0[r, 1]), int(self.rect_vel[r, 1]), i, w - 32)
                out[y:y + 32, x:x + 32] = self.rect_col[r]
        elif self.disturbance == "patches":
            p = self.patch
            fresh = noise.integers(0, 256, size=(self.n_patches, p, p, 3), dtype=np.uint8)
            for k in range(self.n_patches):
                y, x = self.patch_yx[i, k]
                out[y:y + p, x:x + p] = fresh[k]
        else:
            out = self._zoomed(out, float(self.zooms[i]))
            wh, ww = self.win_hw
            y = self._bounce(int(self.win_pos0[0]), int(self.win_vel[0]), i, h - wh)
            x = self._bounce(int(self.win_pos0[1]), int(self.win_vel[1]), i, w - ww)
            out[y:y + wh, x:x + ww] = noise.integers(0, 256, size=(wh, ww, 3), dtype=np.uint8)
        return out


class StreamBatch:
    """S independent streams presented as one batch: ``frame(i)`` -> (S, H, W, 3)."""

    def __init__(self, streams):
        self.streams = list(streams)
        self.n_streams = len(self.streams)
        s0 = self.streams[0]
        self.width, self.height, self.n_frames = s0.width, s0.height, s0.n_frames

    def frame(self, i: int, stream: int | None = None) -> np.ndarray:
        if stream is not None:
            return self.streams[stream].frame(i)
        return np.stack([s.frame(i) for s in self.streams], 0)
