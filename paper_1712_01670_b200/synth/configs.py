"""The five seeded workloads: stream recipe, matcher settings, CNN trunk."""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable

import numpy as np

from . import nets, streams

SEARCH_ES, SEARCH_DS, SEARCH_TSS = 0, 1, 2
DTYPE_FP32, DTYPE_BF16 = 0, 1


@dataclass
class Workload:
    name: str
    index: int
    width: int
    height: int
    n_streams: int
    n_frames: int
    block: int
    range: int
    search: int
    dtype: int
    layers: list
    make_streams: Callable[..., streams.StreamBatch]
    weight_std: float | None = None
    bias_std: float = 0.05
    psnr_db: float = 20.0
    expire_n: int = 10
    seed: int = 0
    extra: dict = field(default_factory=dict)

    def weights(self):
        return nets.random_weights(self.layers, self.seed, std=self.weight_std, bias_std=self.bias_std)

    def streams(self, n_streams: int | None = None, n_frames: int | None = None, first: int = 0) -> streams.StreamBatch:
        """``n_streams`` streams starting at global stream index ``first`` (a stream's pixels depend
        only on its global index, so ranks can render disjoint subsets)."""
        if first:
            return self.make_streams(n_streams or self.n_streams, n_frames or self.n_frames, first)
        return self.make_streams(n_streams or self.n_streams, n_frames or self.n_frames)


def _seed(idx: int) -> int:
    return streams.BASE_SEED + idx


def tiny_single_layer() -> Workload:
    sd = _seed(1)
    return Workload("tiny_single_layer", 1, 64, 64, 1, 2, 8, 8, SEARCH_ES, DTYPE_FP32,
                    nets.single_conv(64, 64),
                    lambda s, f: streams.StreamBatch([streams.ShiftedPair(sd)]),
                    weight_std=0.1, bias_std=0.0, seed=sd)


def small_cnn_stream() -> Workload:
    sd = _seed(2)
    return Workload("small_cnn_stream", 2, 227, 227, 1, 30, 16, 16, SEARCH_DS, DTYPE_FP32,
                    nets.small_cnn(227, 227),
                    lambda s, f, first=0: streams.StreamBatch(
                        [streams.PannedStream(227, 227, f, sd + 1000 * k, max_pan=3, disturbance="rects")
                         for k in range(first, first + s)]),
                    seed=sd)


def alexnet_stream(grouped: bool = False, dtype: int = DTYPE_BF16) -> Workload:
    """Workload 3.  ``grouped``: the trunk with the cited network's two channel groups in layers 2, 4, 5
    (an extra; the stated workload is ungrouped)."""
    sd = _seed(3)
    n_patches = int(np.ceil(0.10 * 227 * 227 / (24 * 24)))
    return Workload("alexnet_stream" + ("_grouped" if grouped else ""), 3, 227, 227, 1, 100, 16, 16, SEARCH_DS, dtype,
                    nets.alexnet_trunk(227, 227, grouped=grouped),
                    lambda s, f, first=0: streams.StreamBatch(
                        [streams.PannedStream(227, 227, f, sd + 1000 * k, max_pan=4, disturbance="patches",
                                              patch=24, n_patches=n_patches) for k in range(first, first + s)]),
                    seed=sd)


def resnet50_stream() -> Workload:
    sd = _seed(4)
    return Workload("resnet50_stream", 4, 224, 224, 1, 300, 16, 24, SEARCH_DS, DTYPE_BF16,
                    nets.resnet50_trunk(224, 224),
                    lambda s, f, first=0: streams.StreamBatch(
                        [streams.PannedStream(224, 224, f, sd + 1000 * k, max_pan=6, disturbance="window",
                                              window_frac=0.15, zoom=0.02) for k in range(first, first + s)]),
                    seed=sd)


def batched_stress(width: int = 1920, height: int = 1080, canvas: int = 2048) -> Workload:
    sd = _seed(5)
    n_patches = int(np.ceil(0.20 * width * height / (64 * 64)))

    def make(s, f, first=0):
        return streams.StreamBatch(
            [streams.PannedStream(width, height, f, sd + 1000 * k, canvas=canvas, max_pan=8,
                                  disturbance="patches", patch=64, n_patches=n_patches)
             for k in range(first, first + s)])

    return Workload("batched_stress", 5, width, height, 32, 60, 16, 32, SEARCH_DS, DTYPE_BF16,
                    nets.vgg16_trunk(224, 224, height, width), make, seed=sd)


WORKLOADS = {
    1: tiny_single_layer,
    2: small_cnn_stream,
    3: alexnet_stream,
    4: resnet50_stream,
    5: batched_stress,
}
