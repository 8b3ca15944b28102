"""``DeepCache``: a small convenience object over the C ABI.

It owns the opaque cache handle and the torch tensors used as outputs; every
method is one call of the library (``binding.dc_*``).  No arithmetic of the
method happens in Python.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B


class _DevView:
    """Exposes a raw device pointer through ``__cuda_array_interface__``."""

    def __init__(self, ptr: int, shape, typestr: str):
        self.__cuda_array_interface__ = dict(shape=tuple(shape), typestr=typestr, data=(ptr, False), version=2)


def device_view(ptr: int, shape, dtype: torch.dtype, device) -> torch.Tensor:
    """A torch tensor aliasing library-owned device memory (no copy)."""
    if dtype == torch.bfloat16:
        return torch.as_tensor(_DevView(ptr, shape, "<i2"), device=device).view(torch.bfloat16)
    typestr = {torch.float32: "<f4", torch.int32: "<i4", torch.uint8: "|u1", torch.int16: "<i2"}[dtype]
    return torch.as_tensor(_DevView(ptr, shape, typestr), device=device)


class DeepCache:
    def __init__(self, width, height, layers, weights, biases, *, n_streams=1, block=10, search_range=8,
                 search=B.DC_SEARCH_DIAMOND, psnr_db=20.0, expire_n=10, dtype=B.DC_FP32, max_regions=0, skip_k=1,
                 region_mode=B.DC_REGIONS_GLOBAL, cache_pool=False, lrn=(1e-4, 0.75, 1.0), device="cuda:0"):
        if not torch.cuda.is_available():
            raise RuntimeError("DeepCache needs a CUDA device; there is no CPU fallback")
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.layers = [dict(l) for l in layers]
        self.cfg = B.dc_config(width=width, height=height, channels=3, n_streams=n_streams, block=block,
                               range=search_range, search=search, skip_k=skip_k, expire_n=expire_n, psnr_db=psnr_db,
                               dtype=dtype, max_regions=max_regions, region_mode=region_mode,
                               cache_pool=int(bool(cache_pool)), lrn_alpha=lrn[0], lrn_beta=lrn[1], lrn_k=lrn[2])
        self.S, self.W, self.H = n_streams, width, height
        self.Gx, self.Gy = -(-width // block), -(-height // block)
        worst = self.Gx * self.Gy if region_mode == B.DC_REGIONS_PER_BLOCK else -(-self.Gx // 2) * self.Gy
        self.max_regions = max_regions if max_regions > 0 else worst
        self.tdtype = torch.bfloat16 if dtype == B.DC_BF16 else torch.float32
        w_dev = [None if w is None else torch.as_tensor(np.ascontiguousarray(w, np.float32)).to(self.device) for w in weights]
        b_dev = [None if b is None else torch.as_tensor(np.ascontiguousarray(b, np.float32)).to(self.device) for b in biases]
        self.handle = B.dc_cache_create(self.cfg, self.layers, w_dev, b_dev)
        del w_dev, b_dev           # the library has made its own copies

    @classmethod
    def from_workload(cls, w, n_streams=None, **kw):
        ws, bs = w.weights()
        args = dict(n_streams=n_streams or w.n_streams, block=w.block, search_range=w.range, search=w.search,
                    psnr_db=w.psnr_db, expire_n=w.expire_n, dtype=w.dtype)
        args.update(kw)
        return cls(w.width, w.height, w.layers, ws, bs, **args)

    def close(self):
        if self.handle is not None:
            B.dc_cache_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- helpers ----------------------------------------------------------
    def out_shape(self, layer=-1):
        l = self.layers[layer]
        return (self.S, l["out_h"], l["out_w"], l["cout"])

    def _frame(self, frame):
        """(S, H, W, 3) uint8 CUDA tensor and its row pitch in bytes."""
        if not isinstance(frame, torch.Tensor):
            frame = torch.as_tensor(np.ascontiguousarray(frame))
        frame = frame.to(self.device)
        if frame.dim() == 3:
            frame = frame[None]
        assert frame.shape == (self.S, self.H, self.W, 3) and frame.dtype == torch.uint8
        return frame.contiguous(), self.W * 3

    # -- the five calls ---------------------------------------------------
    def reset(self):
        B.dc_cache_reset(self.handle)

    def set_key(self, frame):
        f, pitch = self._frame(frame)
        B.dc_cache_set_key(self.handle, f, pitch)
        torch.cuda.current_stream().synchronize()

    def match_blocks(self, frame):
        f, pitch = self._frame(frame)
        d = self.device
        out = dict(mv=torch.empty((self.S, self.Gy, self.Gx, 2), dtype=torch.int16, device=d),
                   sse=torch.empty((self.S, self.Gy, self.Gx), dtype=torch.int32, device=d),
                   matched=torch.empty((self.S, self.Gy, self.Gx), dtype=torch.uint8, device=d),
                   gmv=torch.empty((self.S, 3), dtype=torch.int32, device=d),
                   regions=torch.zeros((self.S, self.max_regions, 6), dtype=torch.int32, device=d),
                   n_regions=torch.empty((self.S,), dtype=torch.int32, device=d))
        B.dc_match_blocks(self.handle, f, pitch, out["mv"], out["sse"], out["matched"], out["gmv"],
                          out["regions"], out["n_regions"])
        torch.cuda.current_stream().synchronize()
        return out

    def propagate_regions(self, regions, n_regions, layer_begin=0, layer_end=None):
        layer_end = len(self.layers) if layer_end is None else layer_end
        out = torch.zeros((layer_end - layer_begin, self.S, self.max_regions, 6), dtype=torch.int32, device=self.device)
        n_out = torch.zeros((layer_end - layer_begin, self.S), dtype=torch.int32, device=self.device)
        B.dc_propagate_regions(self.handle, regions.contiguous(), n_regions.contiguous(), layer_begin, layer_end, out, n_out)
        torch.cuda.current_stream().synchronize()
        return out, n_out

    def conv_partial(self, layer, in_map, prev_out=None, regions=None, n_regions=None):
        out = torch.zeros(self.out_shape(layer), dtype=self.tdtype, device=self.device)
        B.dc_conv_partial(self.handle, layer, in_map.contiguous(), prev_out, regions, n_regions, out)
        torch.cuda.current_stream().synchronize()
        return out

    def infer_frame(self, frame, want_stats=False, want_out=True):
        f, pitch = self._frame(frame)
        out = torch.empty(self.out_shape(-1), dtype=self.tdtype, device=self.device) if want_out else None
        stats = (B.dc_frame_stats * self.S)() if want_stats else None
        B.dc_infer_frame(self.handle, f, pitch, out, stats)
        if want_stats:
            return out, stats
        return out

    # -- inspection -------------------------------------------------------
    def layer_map(self, layer) -> torch.Tensor:
        ptr, _ = B.dc_cache_layer_map(self.handle, layer)
        torch.cuda.current_stream().synchronize()
        return device_view(ptr, self.out_shape(layer), self.tdtype, self.device).clone()

    def layer_regions(self, layer):
        ptr, nptr = B.dc_cache_layer_regions(self.handle, layer)
        torch.cuda.current_stream().synchronize()
        regs = device_view(ptr, (self.S, self.max_regions, 6), torch.int32, self.device).clone()
        n = device_view(nptr, (self.S,), torch.int32, self.device).clone()
        return regs, n

    def status(self) -> int:
        return B.dc_get_status(self.handle)

    def bytes(self) -> int:
        return B.dc_cache_bytes(self.handle)

    def launches(self) -> int:
        return B.dc_cache_launches(self.handle)
