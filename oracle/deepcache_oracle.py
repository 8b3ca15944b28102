"""Python face of the CPU oracle (``deepcache_oracle.c``).

TEST INFRASTRUCTURE ONLY: used by the tests, the smoke check and the
benchmark's CPU-baseline leg.  It never imports, and is never imported by,
the CUDA package.

``OracleCache`` walks one stream through the cache-aware inference of the
paper, step by step, with every intermediate kept for inspection:

  Section 4 Steps 1-5   block search, PSNR test, mean motion, verify, merge
  Section 5 Table 2     region propagation layer by layer
  Section 5 "Reuse"     copy cached conv outputs inside regions, convolve the rest
  Section 5 (expiry)    a full fresh frame every N frames
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "deepcache_oracle.c")
_LIB = os.path.join(_HERE, "libdeepcache_oracle.so")

KIND_CONV, KIND_MAXPOOL, KIND_RELU, KIND_ADD, KIND_CONCAT, KIND_RESIZE_AREA, KIND_LRN, KIND_FC = range(8)
SEARCH_ES, SEARCH_DS, SEARCH_TSS = 0, 1, 2
QUANT_NONE, QUANT_BF16 = 0, 1


class Region(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("x", "y", "w", "h", "sx", "sy")]


class Layer(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("kind", "kh", "kw", "sh", "sw", "ph", "pw", "cin", "cout",
                                         "relu", "in0", "in1", "out_h", "out_w", "groups")]


REGION_DTYPE = np.dtype([(n, "<i4") for n in ("x", "y", "w", "h", "sx", "sy")])


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP) if the library is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        u8p, i16p, u32p, i32p, dp = (C.POINTER(t) for t in (C.c_uint8, C.c_int16, C.c_uint32, C.c_int32, C.c_double))
        rp, lp = C.POINTER(Region), C.POINTER(Layer)
        i, i64, d = C.c_int, C.c_int64, C.c_double
        L.orc_block_sse.restype = C.c_uint64
        L.orc_block_sse.argtypes = [u8p, u8p, i, i, i64, i, i, i, i, i, i]
        L.orc_psnr_limit.restype = C.c_int64
        L.orc_psnr_limit.argtypes = [i64, d]
        L.orc_psnr_pass.restype = i
        L.orc_psnr_pass.argtypes = [C.c_uint64, i64, d]
        L.orc_search.restype = None
        L.orc_search.argtypes = [u8p, u8p, i, i, i64, i, i, i, i16p, u32p]
        L.orc_search_k.restype = None
        L.orc_search_k.argtypes = [u8p, u8p, i, i, i64, i, i, i, i, i16p, u32p]
        L.orc_mean_mv.restype = None
        L.orc_mean_mv.argtypes = [i16p, u32p, i, i, i, d, i32p]
        L.orc_verify.restype = None
        L.orc_verify.argtypes = [u8p, u8p, i, i, i64, i, i, i, i, d, u8p]
        L.orc_merge.restype = i
        L.orc_merge.argtypes = [u8p, i, i, i, i, i, rp]
        L.orc_accept_own.restype = None
        L.orc_accept_own.argtypes = [i16p, u32p, i, i, i, d, u8p]
        L.orc_merge_own.restype = i
        L.orc_merge_own.argtypes = [u8p, i16p, i, i, i, rp]
        L.orc_propagate_layer.restype = None
        L.orc_propagate_layer.argtypes = [lp, i, i, rp, rp, i, rp]
        L.orc_quant.restype = d
        L.orc_quant.argtypes = [d, i]
        L.orc_quant_array.restype = None
        L.orc_quant_array.argtypes = [dp, i64, i]
        L.orc_input_map.restype = None
        L.orc_input_map.argtypes = [u8p, i, i, i64, i, dp]
        L.orc_resize_area.restype = None
        L.orc_resize_area.argtypes = [u8p, i, i, i64, i, i, i, dp]
        L.orc_conv_reuse.restype = None
        L.orc_conv_reuse.argtypes = [dp, i, i, lp, dp, dp, i, dp, rp, i, dp, u8p]
        L.orc_maxpool.restype = None
        L.orc_maxpool.argtypes = [dp, i, i, lp, dp]
        L.orc_add.restype = None
        L.orc_add.argtypes = [dp, dp, i64, i, i, dp]
        L.orc_relu.restype = None
        L.orc_relu.argtypes = [dp, i64, dp]
        _lib = L
    return _lib


def _p(a: np.ndarray, t):
    return a.ctypes.data_as(C.POINTER(t))


def _u8(a):
    a = np.ascontiguousarray(a, dtype=np.uint8)
    return a


def make_layer(d: dict) -> Layer:
    return Layer(**{k: int(d.get(k, 0)) for k, _ in Layer._fields_})       # groups is optional (0 = ungrouped)


# ---------------------------------------------------------------------------
# step functions (numpy in, numpy out)
# ---------------------------------------------------------------------------
def block_sse(cur, prev, x0, y0, bw, bh, dx, dy):
    """SSE of one block pair; None when the displaced block leaves the frame."""
    cur, prev = _u8(cur), _u8(prev)
    H, W = cur.shape[:2]
    v = lib().orc_block_sse(_p(cur, C.c_uint8), _p(prev, C.c_uint8), W, H, W * 3, x0, y0, bw, bh, dx, dy)
    return None if v == 2 ** 64 - 1 else int(v)


def psnr_limit(n: int, T: float) -> int:
    return int(lib().orc_psnr_limit(n, T))


def search(cur, prev, B, R, kind, skip_k=1):
    """Section 4 Step 2.  Returns mv int16 [Gy, Gx, 2] as (dx, dy) and sse uint32 [Gy, Gx].
    skip_k > 1: only blocks on every skip_k-th row and column are searched (the rest: sse = 2^32 - 1)."""
    cur, prev = _u8(cur), _u8(prev)
    H, W = cur.shape[:2]
    Gx, Gy = -(-W // B), -(-H // B)
    mv = np.zeros((Gy, Gx, 2), np.int16)
    sse = np.zeros((Gy, Gx), np.uint32)
    lib().orc_search_k(_p(cur, C.c_uint8), _p(prev, C.c_uint8), W, H, W * 3, B, R, kind, skip_k,
                       _p(mv, C.c_int16), _p(sse, C.c_uint32))
    return mv, sse


def mean_mv(mv, sse, W, H, B, T):
    """Section 4 Step 3.  Returns (Mx, My, K)."""
    out = np.zeros(3, np.int32)
    lib().orc_mean_mv(_p(np.ascontiguousarray(mv), C.c_int16), _p(np.ascontiguousarray(sse), C.c_uint32),
                      W, H, B, T, _p(out, C.c_int32))
    return int(out[0]), int(out[1]), int(out[2])


def verify(cur, prev, B, Mx, My, K, T):
    """Section 4 Step 4.  Returns matched uint8 [Gy, Gx]."""
    cur, prev = _u8(cur), _u8(prev)
    H, W = cur.shape[:2]
    Gx, Gy = -(-W // B), -(-H // B)
    m = np.zeros((Gy, Gx), np.uint8)
    lib().orc_verify(_p(cur, C.c_uint8), _p(prev, C.c_uint8), W, H, W * 3, B, Mx, My, K, T, _p(m, C.c_uint8))
    return m


def merge(matched, W, H, B, Mx, My):
    """Section 4 Step 5.  Returns a structured array of regions ordered by (y, x)."""
    matched = _u8(matched)
    out = np.zeros(matched.size, REGION_DTYPE)
    n = lib().orc_merge(_p(matched, C.c_uint8), W, H, B, Mx, My, out.ctypes.data_as(C.POINTER(Region)))
    return out[:n].copy()


REGIONS_GLOBAL, REGIONS_PER_BLOCK = 0, 1


def accept_own(mv, sse, W, H, B, T):
    """Per-block variant of Step 4: a block is matched when its own best vector passes the PSNR test."""
    mv = np.ascontiguousarray(mv, np.int16)
    sse = np.ascontiguousarray(sse, np.uint32)
    matched = np.zeros(sse.shape, np.uint8)
    lib().orc_accept_own(_p(mv, C.c_int16), _p(sse, C.c_uint32), W, H, B, float(T), _p(matched, C.c_uint8))
    return matched


def merge_own(matched, mv, W, H, B):
    """Per-block variant of Step 5: only neighbours with the same vector merge; each rectangle carries its own."""
    matched = _u8(matched)
    mv = np.ascontiguousarray(mv, np.int16)
    out = np.zeros(matched.size, REGION_DTYPE)
    n = lib().orc_merge_own(_p(matched, C.c_uint8), _p(mv, C.c_int16), W, H, B, out.ctypes.data_as(C.POINTER(Region)))
    return out[:n].copy()


def match_blocks(cur, prev, B, R, kind, T, skip_k=1, region_mode=REGIONS_GLOBAL):
    """Steps 1-5 in order.  Returns dict(mv, sse, M, K, matched, regions)."""
    H, W = cur.shape[:2]
    mv, sse = search(cur, prev, B, R, kind, skip_k)
    Mx, My, K = mean_mv(mv, sse, W, H, B, T)
    if region_mode == REGIONS_PER_BLOCK:
        matched = accept_own(mv, sse, W, H, B, T)
        regions = merge_own(matched, mv, W, H, B)
    else:
        matched = verify(cur, prev, B, Mx, My, K, T)
        regions = merge(matched, W, H, B, Mx, My)
    return dict(mv=mv, sse=sse, M=(Mx, My), K=K, matched=matched, regions=regions)


def propagate_layer(layer: dict, in_h: int, in_w: int, regs0, regs1=None):
    """Table 2 for one layer; slot-preserving (vanished regions become all-zero)."""
    regs0 = np.ascontiguousarray(regs0, REGION_DTYPE)
    regs1 = regs0 if regs1 is None else np.ascontiguousarray(regs1, REGION_DTYPE)
    out = np.zeros(len(regs0), REGION_DTYPE)
    L = make_layer(layer)
    rp = C.POINTER(Region)
    lib().orc_propagate_layer(C.byref(L), in_h, in_w, regs0.ctypes.data_as(rp), regs1.ctypes.data_as(rp),
                              len(regs0), out.ctypes.data_as(rp))
    return out


def _in_shape(layers, idx, frame_hw):
    if idx < 0:
        return frame_hw
    return layers[idx]["out_h"], layers[idx]["out_w"]


def propagate(layers, frame_hw, regions):
    """Region list at the output of every layer (list of structured arrays)."""
    per_layer = []
    for l in layers:
        r0 = regions if l["in0"] < 0 else per_layer[l["in0"]]
        r1 = None
        if l["kind"] in (KIND_ADD, KIND_CONCAT):
            r1 = regions if l["in1"] < 0 else per_layer[l["in1"]]
        ih, iw = _in_shape(layers, l["in0"], frame_hw)
        per_layer.append(propagate_layer(l, ih, iw, r0, r1))
    return per_layer


def quant_array(a: np.ndarray, mode: int) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float64).copy()
    lib().orc_quant_array(_p(a, C.c_double), a.size, mode)
    return a


def input_map(frame, mode):
    frame = _u8(frame)
    H, W = frame.shape[:2]
    out = np.empty((H, W, 3), np.float64)
    lib().orc_input_map(_p(frame, C.c_uint8), W, H, W * 3, mode, _p(out, C.c_double))
    return out


def resize_area(frame, Ho, Wo, mode):
    frame = _u8(frame)
    H, W = frame.shape[:2]
    out = np.empty((Ho, Wo, 3), np.float64)
    lib().orc_resize_area(_p(frame, C.c_uint8), W, H, W * 3, Wo, Ho, mode, _p(out, C.c_double))
    return out


def conv_reuse(x, layer, weight, bias, mode, prev_out=None, regions=None):
    """Section 5 "Reuse" for one conv layer.  Returns (out, reused byte map)."""
    x = np.ascontiguousarray(x, np.float64)
    Hi, Wi = x.shape[:2]
    L = make_layer(layer)
    out = np.empty((L.out_h, L.out_w, L.cout), np.float64)
    reused = np.zeros((L.out_h, L.out_w), np.uint8)
    weight = np.ascontiguousarray(weight, np.float64)
    bias = np.ascontiguousarray(bias, np.float64)
    if prev_out is not None and regions is not None and len(regions):
        regions = np.ascontiguousarray(regions, REGION_DTYPE)
        prev_out = np.ascontiguousarray(prev_out, np.float64)
        pp, rp, n = _p(prev_out, C.c_double), regions.ctypes.data_as(C.POINTER(Region)), len(regions)
    else:
        pp, rp, n = None, None, 0
    lib().orc_conv_reuse(_p(x, C.c_double), Hi, Wi, C.byref(L), _p(weight, C.c_double), _p(bias, C.c_double),
                         mode, pp, rp, n, _p(out, C.c_double), _p(reused, C.c_uint8))
    return out, reused


def maxpool(x, layer):
    x = np.ascontiguousarray(x, np.float64)
    L = make_layer(layer)
    out = np.empty((L.out_h, L.out_w, L.cout), np.float64)
    lib().orc_maxpool(_p(x, C.c_double), x.shape[0], x.shape[1], C.byref(L), _p(out, C.c_double))
    return out


def pool_reuse(x, layer, prev_out=None, regions=None):
    """Section 5 notes that the cache extends to other layer types; this is that extension for max pooling,
    with the three steps of "Reuse": copy the layer's reusable rectangles from the cached pooled map, mark
    them, pool the input only where nothing was copied.  Returns (out, reused byte map)."""
    return _copy_rectangles(maxpool(x, layer), prev_out, regions)


def lrn_reuse(x, layer, alpha, beta, k, mode, prev_out=None, regions=None):
    """The same extension for an LRN layer: cached rectangles copied, the rest normalised from the input."""
    return _copy_rectangles(lrn(x, layer, alpha, beta, k, mode), prev_out, regions)


def _copy_rectangles(out, prev_out, regions):
    reused = np.zeros(out.shape[:2], np.uint8)
    if prev_out is not None and regions is not None:
        for r in regions:
            if r["w"] <= 0 or r["h"] <= 0:
                continue
            y, x0, h, w, sy, sx = (int(r[k]) for k in ("y", "x", "h", "w", "sy", "sx"))
            out[y:y + h, x0:x0 + w] = prev_out[sy:sy + h, sx:sx + w]
            reused[y:y + h, x0:x0 + w] = 1
    return out, reused


def lrn(x, layer, alpha, beta, k, mode):
    """Local response normalisation over a spatial window inside each channel: the form Table 2's LRN row
    describes (a radius r erodes the rectangle by r on every side).  With n = 2 r + 1:
        b[y, x, c] = a[y, x, c] / (k + alpha / n^2 * sum_{|dy|,|dx| <= r} a[y + dy, x + dx, c]^2) ^ beta
    pixels outside the map count as zero; the divisor n^2 is the same at the borders.  r = layer's ph."""
    x = np.ascontiguousarray(x, np.float64)
    r = int(layer["ph"])
    n = 2 * r + 1
    H, W, _ = x.shape
    sq = np.zeros((H + 2 * r, W + 2 * r, x.shape[2]), np.float64)
    sq[r:r + H, r:r + W] = x * x
    total = np.zeros_like(x)
    for dy in range(n):
        for dx in range(n):
            total += sq[dy:dy + H, dx:dx + W]
    out = x / (k + alpha / (n * n) * total) ** beta
    return quant_array(out, mode)


def concat(a, b):
    """Channel concatenation (Table 2's Concat row, two inputs): the channels of a, then those of b."""
    return np.concatenate([np.asarray(a, np.float64), np.asarray(b, np.float64)], axis=2)


def fully_connected(x, layer, weight, bias, mode):
    """A fully-connected layer on an H x W x C map is the convolution whose kernel covers the whole map without
    padding (one output pixel); weight is [cout][H][W][cin].  Table 2: nothing of its output is reusable."""
    L = dict(layer, kind=KIND_CONV, kh=x.shape[0], kw=x.shape[1], sh=1, sw=1, ph=0, pw=0, out_h=1, out_w=1)
    out, _ = conv_reuse(x, L, weight, bias, mode)
    return out


def add(a, b, relu, mode):
    """Residual add (a multi-input layer of Table 2): element-wise sum, optional ReLU, storage rounding."""
    a = np.ascontiguousarray(a, np.float64)
    b = np.ascontiguousarray(b, np.float64)
    out = np.empty_like(a)
    lib().orc_add(_p(a, C.c_double), _p(b, C.c_double), a.size, relu, mode, _p(out, C.c_double))
    return out


def relu(a):
    """A stand-alone ReLU layer (Table 2, "others": the rectangle passes unchanged).  max(a, 0) of a stored value
    is a stored value, so there is no rounding step."""
    a = np.ascontiguousarray(a, np.float64)
    out = np.empty_like(a)
    lib().orc_relu(_p(a, C.c_double), a.size, _p(out, C.c_double))
    return out


# ---------------------------------------------------------------------------
# one stream, frame after frame
# ---------------------------------------------------------------------------
class OracleCache:
    """Cache-aware inference of one video stream, following the paper's order.

    ``infer_frame(frame)`` returns a dict with the output map and everything
    decided along the way.  ``use_cache=False`` gives the no-cache baseline of
    Section 7 (plain full inference of every frame).
    """

    def __init__(self, width, height, layers, weights, biases, *, block=10, search_range=8,
                 search_kind=SEARCH_DS, psnr_db=20.0, expire_n=10, quant=QUANT_NONE, use_cache=True, skip_k=1,
                 region_mode=0, cache_pool=False, lrn=(1e-4, 0.75, 1.0)):
        self.W, self.H = width, height
        self.layers = layers
        self.block, self.R, self.kind = block, search_range, search_kind
        self.T, self.N, self.quant, self.use_cache = psnr_db, expire_n, quant, use_cache
        self.skip_k, self.region_mode, self.cache_pool = skip_k, region_mode, cache_pool
        self.lrn = lrn                 # (alpha, beta, k) of every LRN layer
        # weights are stored at the storage precision (bf16 workloads round them once)
        self.weights = [None if w is None else quant_array(w, quant) for w in weights]
        self.biases = [None if b is None else np.asarray(b, np.float64) for b in biases]
        self.reset()

    def reset(self):
        """Forget the cache: the next frame is computed in full."""
        self.frame_idx = 0
        self.prev_frame = None
        self.prev_maps = None          # per layer: cached conv output of the last frame

    def infer_frame(self, frame):
        frame = _u8(frame)
        layers = self.layers
        # Section 5: every N-th frame is computed from scratch, cache rewritten
        refresh = (not self.use_cache) or self.prev_frame is None or (self.frame_idx % self.N == 0)
        info = dict(refreshed=bool(refresh), match=None, regions=None, reused=[None] * len(layers))
        per_layer_regions = None
        if not refresh:
            m = match_blocks(frame, self.prev_frame, self.block, self.R, self.kind, self.T, self.skip_k,
                             self.region_mode)
            per_layer_regions = propagate(layers, (self.H, self.W), m["regions"])
            info["match"], info["regions"] = m, per_layer_regions
        maps = []
        net_in = None
        for i, l in enumerate(layers):
            k = l["kind"]
            if l["in0"] < 0 and k != KIND_RESIZE_AREA:
                if net_in is None:
                    net_in = input_map(frame, self.quant)
                x = net_in
            elif k != KIND_RESIZE_AREA:
                x = maps[l["in0"]]
            if k == KIND_CONV:
                prev = None if refresh else self.prev_maps[i]
                regs = None if refresh else per_layer_regions[i]
                out, reused = conv_reuse(x, l, self.weights[i], self.biases[i], self.quant, prev, regs)
                info["reused"][i] = reused
            elif k == KIND_MAXPOOL:
                if self.cache_pool and not refresh:
                    out, reused = pool_reuse(x, l, self.prev_maps[i], per_layer_regions[i])
                    info["reused"][i] = reused
                else:
                    out = maxpool(x, l)
            elif k == KIND_ADD:
                out = add(x, maps[l["in1"]], l["relu"], self.quant)
            elif k == KIND_RESIZE_AREA:
                assert l["in0"] < 0, "area resize reads the input frame"
                out = resize_area(frame, l["out_h"], l["out_w"], self.quant)
            elif k == KIND_RELU:
                out = relu(x)
            elif k == KIND_LRN:
                if self.cache_pool and not refresh:
                    out, reused = lrn_reuse(x, l, *self.lrn, self.quant, self.prev_maps[i], per_layer_regions[i])
                    info["reused"][i] = reused
                else:
                    out = lrn(x, l, *self.lrn, self.quant)
            elif k == KIND_CONCAT:
                out = concat(x, maps[l["in1"]])
            elif k == KIND_FC:
                out = fully_connected(x, l, self.weights[i], self.biases[i], self.quant)
            else:
                raise ValueError(f"layer kind {k} has no execution rule in the oracle")
            maps.append(out)
        # the frame becomes the next key, the conv outputs the next values (Section 3)
        self.prev_frame = frame.copy()
        kept = (KIND_CONV, KIND_MAXPOOL, KIND_LRN) if self.cache_pool else (KIND_CONV,)
        self.prev_maps = [m if layers[i]["kind"] in kept else None for i, m in enumerate(maps)]
        self.frame_idx += 1
        info["maps"] = maps
        info["out"] = maps[-1]
        return info
