"""Thin ctypes binding of ``libdeepcache.so`` (see ``include/deepcache.h``).

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  torch supplies device memory and the CUDA stream.  There is no CPU
fallback: if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

DC_MAX_LAYERS = 128
DC_OK = 0
DC_ERR_ARG, DC_ERR_CONFIG, DC_ERR_ALLOC, DC_ERR_CUDA, DC_ERR_OVERFLOW, DC_ERR_TIMEOUT, DC_ERR_STATE, DC_ERR_LIMIT = range(-1, -9, -1)
DC_NOALLOC_MAX_STREAMS = 64
DC_CONV, DC_MAXPOOL, DC_RELU, DC_ADD, DC_CONCAT, DC_RESIZE_AREA, DC_LRN, DC_FC = range(8)
DC_SEARCH_EXHAUSTIVE, DC_SEARCH_DIAMOND, DC_SEARCH_THREE_STEP = 0, 1, 2
DC_REGIONS_GLOBAL, DC_REGIONS_PER_BLOCK = 0, 1
DC_FP32, DC_BF16 = 0, 1

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libdeepcache.so")


class dc_region(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("x", "y", "w", "h", "sx", "sy")]


class dc_layer_desc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("kind", "kh", "kw", "sh", "sw", "ph", "pw", "cin", "cout",
                                         "relu", "in0", "in1", "out_h", "out_w", "groups")]


class dc_config(C.Structure):
    _fields_ = [("width", C.c_int32), ("height", C.c_int32), ("channels", C.c_int32), ("n_streams", C.c_int32),
                ("block", C.c_int32), ("range", C.c_int32), ("search", C.c_int32), ("skip_k", C.c_int32),
                ("expire_n", C.c_int32), ("psnr_db", C.c_double), ("dtype", C.c_int32), ("max_regions", C.c_int32),
                ("region_mode", C.c_int32), ("cache_pool", C.c_int32),
                ("lrn_alpha", C.c_double), ("lrn_beta", C.c_double), ("lrn_k", C.c_double)]


class dc_frame_stats(C.Structure):
    _fields_ = [("refreshed", C.c_int32), ("n_blocks", C.c_int32), ("k_passed", C.c_int32), ("mvx", C.c_int32),
                ("mvy", C.c_int32), ("n_matched", C.c_int32), ("n_regions", C.c_int32),
                ("reuse_ratio", C.c_float * DC_MAX_LAYERS)]


REGION_DTYPE = np.dtype([(n, "<i4") for n in ("x", "y", "w", "h", "sx", "sy")])

EXPORTS = ["dc_cache_create", "dc_cache_destroy", "dc_cache_reset", "dc_cache_bytes", "dc_cache_set_key",
           "dc_match_blocks", "dc_propagate_regions", "dc_conv_partial", "dc_infer_frame", "dc_infer_frame_host",
           "dc_prefetch_frame_host", "dc_lookahead_frame",
           "dc_cache_layer_map", "dc_cache_layer_regions", "dc_cache_layer_conv_scheme", "dc_get_status", "dc_cache_launches",
           "dc_cache_set_profiling", "dc_cache_profile", "dc_cache_counters", "dc_search_blocks_noalloc", "dc_strerror"]
PROFILE_STAGES = ["search", "verify", "merge", "propagate", "classify_copy", "conv", "input", "pointwise", "key_update"]

_lib = None


class DeepCacheError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {strerror(status)} ({status})")


def load():
    """Loads the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(f"{_LIB_PATH} not found: build it with `python -m paper_1712_01670_b200.build` "
                              "(there is no CPU fallback)")
        L = C.CDLL(_LIB_PATH)
        vp, i, sz = C.c_void_p, C.c_int, C.c_size_t
        L.dc_cache_create.argtypes = [C.POINTER(dc_config), C.POINTER(dc_layer_desc), i, C.POINTER(vp), C.POINTER(vp), vp, C.POINTER(vp)]
        L.dc_cache_destroy.argtypes = [vp]
        L.dc_cache_reset.argtypes = [vp]
        L.dc_cache_bytes.argtypes = [vp, C.POINTER(sz)]
        L.dc_cache_set_key.argtypes = [vp, vp, sz]
        L.dc_match_blocks.argtypes = [vp, vp, sz, vp, vp, vp, vp, vp, vp]
        L.dc_propagate_regions.argtypes = [vp, vp, vp, i, i, vp, vp]
        L.dc_conv_partial.argtypes = [vp, i, vp, vp, vp, vp, vp]
        L.dc_infer_frame.argtypes = [vp, vp, sz, vp, C.POINTER(dc_frame_stats)]
        L.dc_infer_frame_host.argtypes = [vp, vp, sz, vp, C.POINTER(dc_frame_stats)]
        L.dc_prefetch_frame_host.argtypes = [vp, vp, sz]
        L.dc_lookahead_frame.argtypes = [vp, vp, sz]
        L.dc_cache_layer_map.argtypes = [vp, i, C.POINTER(vp), C.POINTER(sz)]
        L.dc_cache_layer_regions.argtypes = [vp, i, C.POINTER(vp), C.POINTER(vp)]
        L.dc_cache_layer_conv_scheme.argtypes = [vp, i, C.POINTER(C.c_int32)]
        L.dc_get_status.argtypes = [vp, C.POINTER(C.c_int32)]
        L.dc_cache_launches.argtypes = [vp, C.POINTER(C.c_int64)]
        L.dc_cache_set_profiling.argtypes = [vp, i]
        L.dc_cache_profile.argtypes = [vp, C.POINTER(C.c_float), C.POINTER(C.c_int64)]
        L.dc_cache_counters.argtypes = [vp, C.POINTER(C.c_int64), C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
        L.dc_search_blocks_noalloc.argtypes = [vp, vp, sz, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                               C.c_int32, C.c_double, vp, vp, vp, vp]
        L.dc_strerror.argtypes = [i]
        L.dc_strerror.restype = C.c_char_p
        for name in EXPORTS[:-1]:
            getattr(L, name).restype = i
        _lib = L
    return _lib


def strerror(status: int) -> str:
    return load().dc_strerror(status).decode()


def _check(rc: int, where: str):
    if rc != DC_OK:
        raise DeepCacheError(rc, where)


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        assert t.is_cuda and t.is_contiguous()
        return C.c_void_p(t.data_ptr())
    return C.c_void_p(int(t))


def make_layers(layers) -> C.Array:
    arr = (dc_layer_desc * len(layers))()
    for k, l in enumerate(layers):
        for name, _ in dc_layer_desc._fields_:
            setattr(arr[k], name, int(l.get(name, 0)) if name == "groups" else int(l[name]))
    return arr


# --------------------------------------------------------------------------
# the C entry points, same names, torch tensors for device memory
# --------------------------------------------------------------------------
def dc_cache_create(cfg: dc_config, layers, weights, biases, stream=None):
    """weights / biases: per layer a float32 CUDA tensor ([cout, kh, kw, cin] / [cout]) or None."""
    n = len(layers)
    arr = make_layers(layers)
    wp, bp = (C.c_void_p * n)(), (C.c_void_p * n)()
    for k in range(n):
        wp[k] = weights[k].data_ptr() if weights[k] is not None else None
        bp[k] = biases[k].data_ptr() if biases[k] is not None else None
    out = C.c_void_p()
    st = stream if stream is not None else torch.cuda.current_stream().cuda_stream
    _check(load().dc_cache_create(C.byref(cfg), arr, n, wp, bp, C.c_void_p(st), C.byref(out)), "dc_cache_create")
    return out


def dc_cache_destroy(cache):
    _check(load().dc_cache_destroy(cache), "dc_cache_destroy")


def dc_cache_reset(cache):
    _check(load().dc_cache_reset(cache), "dc_cache_reset")


def dc_cache_bytes(cache) -> int:
    v = C.c_size_t()
    _check(load().dc_cache_bytes(cache, C.byref(v)), "dc_cache_bytes")
    return v.value


def dc_cache_launches(cache) -> int:
    v = C.c_int64()
    _check(load().dc_cache_launches(cache, C.byref(v)), "dc_cache_launches")
    return v.value


def dc_cache_set_key(cache, frame, pitch):
    _check(load().dc_cache_set_key(cache, _ptr(frame), pitch), "dc_cache_set_key")


def dc_match_blocks(cache, frame, pitch, block_mv=None, block_sse=None, matched=None, global_mv=None,
                    regions=None, n_regions=None):
    _check(load().dc_match_blocks(cache, _ptr(frame), pitch, _ptr(block_mv), _ptr(block_sse), _ptr(matched),
                                  _ptr(global_mv), _ptr(regions), _ptr(n_regions)), "dc_match_blocks")


def dc_propagate_regions(cache, regions_in, n_in, layer_begin, layer_end, regions_out, n_out=None):
    _check(load().dc_propagate_regions(cache, _ptr(regions_in), _ptr(n_in), layer_begin, layer_end,
                                       _ptr(regions_out), _ptr(n_out)), "dc_propagate_regions")


def dc_conv_partial(cache, layer, in_map, prev_out, regions, n_regions, out_map):
    _check(load().dc_conv_partial(cache, layer, _ptr(in_map), _ptr(prev_out), _ptr(regions), _ptr(n_regions),
                                  _ptr(out_map)), "dc_conv_partial")


def dc_infer_frame(cache, frame, pitch, out_map=None, stats=None):
    _check(load().dc_infer_frame(cache, _ptr(frame), pitch, _ptr(out_map), stats), "dc_infer_frame")


def dc_infer_frame_host(cache, frame_host_ptr, pitch, out_host_ptr=None, stats=None):
    _check(load().dc_infer_frame_host(cache, C.c_void_p(frame_host_ptr), pitch,
                                      C.c_void_p(out_host_ptr) if out_host_ptr else None, stats), "dc_infer_frame_host")


def dc_lookahead_frame(cache, frame, pitch):
    _check(load().dc_lookahead_frame(cache, _ptr(frame), pitch), "dc_lookahead_frame")


def dc_prefetch_frame_host(cache, frame_host_ptr, pitch):
    _check(load().dc_prefetch_frame_host(cache, C.c_void_p(frame_host_ptr), pitch), "dc_prefetch_frame_host")


def dc_cache_layer_map(cache, layer):
    p, n = C.c_void_p(), C.c_size_t()
    _check(load().dc_cache_layer_map(cache, layer, C.byref(p), C.byref(n)), "dc_cache_layer_map")
    return p.value, n.value


def dc_cache_layer_regions(cache, layer):
    p, n = C.c_void_p(), C.c_void_p()
    _check(load().dc_cache_layer_regions(cache, layer, C.byref(p), C.byref(n)), "dc_cache_layer_regions")
    return p.value, n.value


def dc_cache_layer_conv_scheme(cache, layer: int) -> int:
    v = C.c_int32(0)
    _check(load().dc_cache_layer_conv_scheme(cache, layer, C.byref(v)), "dc_cache_layer_conv_scheme")
    return v.value


def dc_get_status(cache) -> int:
    v = C.c_int32()
    _check(load().dc_get_status(cache, C.byref(v)), "dc_get_status")
    return v.value


def dc_cache_set_profiling(cache, enable: bool):
    _check(load().dc_cache_set_profiling(cache, int(enable)), "dc_cache_set_profiling")


def dc_cache_profile(cache):
    """{stage: (milliseconds, launches)} recorded since the last call."""
    ms = (C.c_float * len(PROFILE_STAGES))()
    n = (C.c_int64 * len(PROFILE_STAGES))()
    _check(load().dc_cache_profile(cache, ms, n), "dc_cache_profile")
    return {name: (float(ms[k]), int(n[k])) for k, name in enumerate(PROFILE_STAGES)}


def dc_cache_counters(cache, n_layers: int):
    """(reused pixels per layer, frames served from cache, full fresh frames) since the last reset."""
    px = (C.c_int64 * n_layers)()
    a, b = C.c_int64(), C.c_int64()
    _check(load().dc_cache_counters(cache, px, C.byref(a), C.byref(b)), "dc_cache_counters")
    return [int(v) for v in px], a.value, b.value


def dc_search_blocks_noalloc(frame, prev, pitch, width, height, n_streams, block, search_range, search, psnr_db,
                             block_mv, block_sse, global_mv, stream=None):
    """Block search for callers that cannot allocate device memory: no cache handle, the only scratch
    is a fixed array inside the library.  Calls on one GPU must not overlap (they share that array)."""
    st = stream if stream is not None else torch.cuda.current_stream().cuda_stream
    _check(load().dc_search_blocks_noalloc(_ptr(frame), _ptr(prev), pitch, width, height, n_streams, block,
                                           search_range, search, psnr_db, _ptr(block_mv), _ptr(block_sse),
                                           _ptr(global_mv), C.c_void_p(st)), "dc_search_blocks_noalloc")
