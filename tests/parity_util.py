"""Helpers shared by the GPU parity tests: run the CUDA path and the oracle side by side."""
import numpy as np
import torch

from oracle import deepcache_oracle as orc
from paper_1712_01670_b200 import binding as B
from paper_1712_01670_b200.engine import DeepCache
from paper_1712_01670_b200.synth import configs

FP32_MAX_ABS = 1e-4        # feature maps, float32 networks: max |a - b|
BF16_REL = 2e-2            # feature maps, bfloat16 networks: max |a - b| / max |b|


def regions_np(t: torch.Tensor) -> np.ndarray:
    """(n, 6) int32 tensor -> structured array comparable with the oracle's."""
    a = np.ascontiguousarray(t.cpu().numpy().astype(np.int32))
    return a.view(orc.REGION_DTYPE).reshape(-1)


def assert_regions_equal(got, want, what=""):
    got, want = np.asarray(got), np.asarray(want)
    assert len(got) == len(want), f"{what}: {len(got)} rectangles, oracle has {len(want)}"
    for name in orc.REGION_DTYPE.names:
        assert np.array_equal(got[name], want[name]), f"{what}: field {name} differs"


def assert_match_equal(gpu: dict, s: int, m: dict, what=""):
    """gpu: output of DeepCache.match_blocks; m: oracle match_blocks dict for stream s."""
    assert np.array_equal(gpu["mv"][s].cpu().numpy(), m["mv"]), f"{what}: block motion vectors differ"
    assert np.array_equal(gpu["sse"][s].cpu().numpy().view(np.uint32), m["sse"]), f"{what}: block SSE differ"
    assert tuple(gpu["gmv"][s].cpu().tolist()) == (m["M"][0], m["M"][1], m["K"]), f"{what}: global motion differs"
    assert np.array_equal(gpu["matched"][s].cpu().numpy(), m["matched"]), f"{what}: matched map differs"
    n = int(gpu["n_regions"][s])
    assert_regions_equal(regions_np(gpu["regions"][s, :n]), m["regions"], what)


def map_error(got: torch.Tensor, want: np.ndarray, bf16: bool) -> float:
    g = got.float().cpu().numpy().astype(np.float64)
    assert g.shape == want.shape, (g.shape, want.shape)
    err = np.abs(g - want).max()
    if bf16:
        return float(err / max(np.abs(want).max(), 1e-30))
    return float(err)


def assert_map_close(got, want, bf16, what=""):
    e = map_error(got, want, bf16)
    tol = BF16_REL if bf16 else FP32_MAX_ABS
    assert e <= tol, f"{what}: error {e:.3e} exceeds {tol:.1e}"
    return e


def assert_map_close_per_element(got, want, what=""):
    """bfloat16 maps, element by element: |a - b| <= 2e-2 |b| + 2e-2 max|b| / 64.  The per-map bound above would let a
    channel of small magnitude be far off; this one does not.  Meant for a single layer fed the same stored input
    on both sides, where only the accumulation order and the final rounding differ."""
    g = got.float().cpu().numpy().astype(np.float64)
    assert g.shape == want.shape, (g.shape, want.shape)
    bound = BF16_REL * np.abs(want) + BF16_REL * np.abs(want).max() / 64.0
    excess = np.abs(g - want) - bound
    assert excess.max() <= 0.0, f"{what}: element {np.unravel_index(excess.argmax(), excess.shape)} off by {np.abs(g - want).flat[excess.argmax()]:.3e}"


class CroppedStreams:
    """A stream batch cut to the top-left h x w pixels of every frame."""

    def __init__(self, batch, h, w):
        self.batch, self.h, self.w = batch, h, w

    def frame(self, i, s=None):
        f = self.batch.frame(i) if s is None else self.batch.frame(i, s)
        return np.ascontiguousarray(f[..., :self.h, :self.w, :])


def crop_workload(w, height, width):
    """Makes workload ``w`` deliver frames of height x width (the top-left corner of its own frames)."""
    inner = w.make_streams
    w.make_streams = lambda s, f, first=0: CroppedStreams(inner(s, f, first) if first else inner(s, f), height, width)
    w.width, w.height = width, height
    return w


def make_oracles(w, n_streams, **kw):
    ws, bs = w.weights()
    quant = orc.QUANT_BF16 if w.dtype == configs.DTYPE_BF16 else orc.QUANT_NONE
    args = dict(block=w.block, search_range=w.range, search_kind=w.search, psnr_db=w.psnr_db,
                expire_n=w.expire_n, quant=quant)
    args.update(kw)
    return [orc.OracleCache(w.width, w.height, w.layers, ws, bs, **args) for _ in range(n_streams)]


def run_stream_parity(w, n_streams, frame_ids, check_layers=True, **kw):
    """Feeds the same frames to the CUDA path and to one oracle per stream; checks every frame:
    bit-exact matcher outputs, rectangles at every layer and reuse ratios, maps within tolerance."""
    bf16 = w.dtype == configs.DTYPE_BF16
    sb = w.streams(n_streams, max(frame_ids) + 1)
    dc = DeepCache.from_workload(w, n_streams=n_streams, **{k: v for k, v in kw.items() if k in ("expire_n", "skip_k", "region_mode", "cache_pool")})
    oracles = make_oracles(w, n_streams, **kw)
    worst = 0.0
    try:
        for fi in frame_ids:
            frames = sb.frame(fi)
            out, stats = dc.infer_frame(frames, want_stats=True)
            for s in range(n_streams):
                o = oracles[s].infer_frame(frames[s])
                what = f"{w.name} frame {fi} stream {s}"
                assert bool(stats[s].refreshed) == o["refreshed"], what
                if not o["refreshed"]:
                    m = o["match"]
                    assert (stats[s].mvx, stats[s].mvy, stats[s].k_passed) == (m["M"][0], m["M"][1], m["K"]), what
                    assert stats[s].n_matched == int(m["matched"].sum()), what
                    assert stats[s].n_regions == len(m["regions"]), what
                    n = len(m["regions"])
                    regs0, _ = dc.layer_regions(-1)
                    assert_regions_equal(regions_np(regs0[s, :n]), m["regions"], what + " frame rectangles")
                    for li, l in enumerate(w.layers):
                        regs, _ = dc.layer_regions(li)
                        assert_regions_equal(regions_np(regs[s, :n]), o["regions"][li], what + f" layer {li}")
                        if l["kind"] == orc.KIND_CONV or (kw.get("cache_pool") and l["kind"] in (orc.KIND_MAXPOOL, orc.KIND_LRN)):
                            want_ratio = float(o["reused"][li].mean())
                            assert abs(stats[s].reuse_ratio[li] - want_ratio) < 1e-6, what + f" layer {li} reuse"
                if check_layers:
                    for li in range(len(w.layers)):
                        e = assert_map_close(dc.layer_map(li)[s], o["maps"][li], bf16, what + f" layer {li}")
                        worst = max(worst, e)
                e = assert_map_close(out[s], o["out"], bf16, what + " output")
                worst = max(worst, e)
            assert dc.status() == B.DC_OK
    finally:
        dc.close()
    return worst
