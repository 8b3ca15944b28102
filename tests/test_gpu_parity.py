"""GPU parity: every C-ABI call against the CPU oracle on the same seeded inputs.

Integer results (motion vectors, SSE, matched maps, rectangles at every layer) must be
bit-exact; feature maps within 1e-4 max-abs (float32) or 2e-2 relative (bfloat16).
"""
import numpy as np
import pytest
import torch

from oracle import deepcache_oracle as orc
from paper_1712_01670_b200 import binding as B
from paper_1712_01670_b200.engine import DeepCache
from paper_1712_01670_b200.synth import configs, nets

import parity_util as U

pytestmark = pytest.mark.gpu


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def matcher_only(width, height, n_streams, block, R, search, psnr_db=20.0, skip_k=1, region_mode=0):
    layers = nets.single_conv(height, width)
    ws, bs = nets.random_weights(layers, 1)
    return DeepCache(width, height, layers, ws, bs, n_streams=n_streams, block=block, search_range=R,
                     search=search, psnr_db=psnr_db, skip_k=skip_k, region_mode=region_mode)


def check_pairs(pairs, block, R, search, psnr_db=20.0, skip_k=1, region_mode=0):
    """pairs: list of (prev, cur) frames of equal size, run as one batch of streams."""
    H, W = pairs[0][0].shape[:2]
    dc = matcher_only(W, H, len(pairs), block, R, search, psnr_db, skip_k, region_mode)
    try:
        dc.set_key(np.stack([p for p, _ in pairs]))
        got = dc.match_blocks(np.stack([c for _, c in pairs]))
        for s, (prev, cur) in enumerate(pairs):
            U.assert_match_equal(got, s, orc.match_blocks(cur, prev, block, R, search, psnr_db, skip_k, region_mode),
                                 f"stream {s}")
        assert dc.status() == B.DC_OK
    finally:
        dc.close()


# ------------------------------------------------------------------ dc_match_blocks
def test_match_workload_1_exhaustive():
    w = configs.WORKLOADS[1]()
    sp = w.streams()
    check_pairs([(sp.frame(0)[0], sp.frame(1)[0])], 8, 8, B.DC_SEARCH_EXHAUSTIVE)


@pytest.mark.parametrize("widx,frames", [(2, (1, 2, 5, 9)), (3, (1, 4, 7)), (4, (1, 2, 3))])
def test_match_diamond_streams(widx, frames):
    w = configs.WORKLOADS[widx]()
    sb = w.streams(1, max(frames) + 1)
    check_pairs([(sb.frame(i - 1)[0], sb.frame(i)[0]) for i in frames], w.block, w.range, B.DC_SEARCH_DIAMOND)


@pytest.mark.parametrize("search", [B.DC_SEARCH_EXHAUSTIVE, B.DC_SEARCH_DIAMOND, B.DC_SEARCH_THREE_STEP])
@pytest.mark.parametrize("block,shape", [(8, (40, 56)), (10, (61, 47)), (16, (16, 16)), (16, (90, 131)), (32, (70, 100)), (5, (23, 29))])
def test_match_edge_geometry(search, block, shape):
    g = rng(block * 7 + shape[0])
    H, W = shape
    prev = g.integers(0, 256, size=(H, W, 3), dtype=np.uint8)
    moved = np.roll(prev, (2, -3), axis=(0, 1))
    moved[H // 3:H // 3 + 9, W // 4:W // 4 + 11] = g.integers(0, 256, size=(min(9, H - H // 3), min(11, W - W // 4), 3))
    smooth = np.clip(prev.astype(np.int32) + g.integers(-6, 7, size=prev.shape), 0, 255).astype(np.uint8)
    const = np.full_like(prev, 93)
    pairs = [(prev, moved), (prev, prev), (prev, smooth), (const, const), (const, prev)]
    check_pairs(pairs, block, 4, search)


def test_match_ties_and_thresholds():
    # periodic pattern: several displacements tie at SSE 0; the smallest motion must win on both sides
    x = np.arange(64)
    row = ((x % 4) * 60).astype(np.uint8)
    prev = np.repeat(np.repeat(row[None, :, None], 48, 0), 3, 2)
    cur = np.roll(prev, -1, axis=1)
    for search in (B.DC_SEARCH_EXHAUSTIVE, B.DC_SEARCH_DIAMOND, B.DC_SEARCH_THREE_STEP):
        check_pairs([(prev, cur), (cur, prev)], 8, 6, search)
    # other thresholds move the integer SSE bound
    g = rng(3)
    a = g.integers(0, 256, size=(48, 64, 3), dtype=np.uint8)
    b = np.clip(a.astype(np.int32) + g.integers(-40, 41, size=a.shape), 0, 255).astype(np.uint8)
    for T in (12.0, 18.5, 25.0, 33.3):
        check_pairs([(a, b)], 8, 3, B.DC_SEARCH_DIAMOND, psnr_db=T)


def test_match_full_hd_batch():
    """Workload 5's matcher geometry (1920x1080, block 16, range 32, last block row 8 px) on 2 streams."""
    w = configs.WORKLOADS[5]()
    sb = w.streams(2, 3)
    pairs = [(sb.frame(1, s), sb.frame(2, s)) for s in range(2)]
    check_pairs(pairs, 16, 32, B.DC_SEARCH_DIAMOND)
    # k-skip at this size: every searched block is walked with a private window from its start
    check_pairs(pairs, 16, 32, B.DC_SEARCH_DIAMOND, skip_k=2)


@pytest.mark.parametrize("widx,frames,R", [(2, (1, 2, 5), 16), (3, (1, 4), 7), (4, (2, 3), 24), (2, (3,), 1)])
def test_match_three_step_streams(widx, frames, R):
    """Three step search (Section 7.5) as the Step 2 unit: first steps 8, 4, 8 and 1 for these ranges."""
    w = configs.WORKLOADS[widx]()
    sb = w.streams(1, max(frames) + 1)
    check_pairs([(sb.frame(i - 1)[0], sb.frame(i)[0]) for i in frames], w.block, R, B.DC_SEARCH_THREE_STEP)
    check_pairs([(sb.frame(i - 1)[0], sb.frame(i)[0]) for i in frames], 10, R, B.DC_SEARCH_THREE_STEP, skip_k=2)


def test_match_three_step_full_hd():
    w = configs.WORKLOADS[5]()
    sb = w.streams(2, 3)
    check_pairs([(sb.frame(1, s), sb.frame(2, s)) for s in range(2)], 16, 32, B.DC_SEARCH_THREE_STEP)


def test_infer_with_three_step():
    w = configs.WORKLOADS[3]()
    w.search = configs.SEARCH_TSS
    U.run_stream_parity(w, 1, list(range(4)))


@pytest.mark.parametrize("R,shape", [(32, (97, 150)), (16, (64, 64)), (8, (50, 300)), (5, (33, 47)), (13, (80, 131)), (0, (32, 32))])
def test_match_exhaustive_16_fast_path(R, shape):
    """16-pixel blocks with exhaustive search run on the register-blocked kernel (full groups of 32 dx values,
    the remaining columns one candidate per lane) and clipped edge blocks on the generic one."""
    g = rng(R * 31 + shape[0])
    H, W = shape
    prev = g.integers(0, 256, size=(H, W, 3), dtype=np.uint8)
    moved = np.roll(prev, (min(R, 3), -min(R, 7)), axis=(0, 1))
    far = np.roll(prev, (-R, R), axis=(0, 1))                  # best vectors at the corner of the range
    smooth = np.clip(prev.astype(np.int32) + g.integers(-6, 7, size=prev.shape), 0, 255).astype(np.uint8)
    const = np.full_like(prev, 200)
    check_pairs([(prev, moved), (prev, far), (prev, smooth), (const, const), (far, prev)], 16, R, B.DC_SEARCH_EXHAUSTIVE)
    check_pairs([(prev, moved)], 16, R, B.DC_SEARCH_EXHAUSTIVE, skip_k=2)


def test_match_exhaustive_video_streams():
    w = configs.WORKLOADS[2]()
    sb = w.streams(1, 4)
    check_pairs([(sb.frame(i - 1)[0], sb.frame(i)[0]) for i in (1, 2, 3)], 16, 16, B.DC_SEARCH_EXHAUSTIVE)
    w = configs.WORKLOADS[5]()                                 # 1920x1080: 120 full columns, last block row 8 px
    sb = w.streams(1, 3)
    f1, f2 = sb.frame(1, 0), sb.frame(2, 0)
    check_pairs([(f1[:200, :1000], f2[:200, :1000])], 16, 32, B.DC_SEARCH_EXHAUSTIVE)


def two_motion_pair(g, H, W):
    prev = g.integers(0, 256, size=(H, W, 3), dtype=np.uint8)
    cur = prev.copy()
    cur[:, W // 2:] = np.roll(prev, (-2, 3), axis=(0, 1))[:, W // 2:]
    cur[H // 3:H // 3 + 7, 2:13] = g.integers(0, 256, size=(7, 11, 3))
    return prev, cur


@pytest.mark.parametrize("search", [B.DC_SEARCH_EXHAUSTIVE, B.DC_SEARCH_DIAMOND, B.DC_SEARCH_THREE_STEP])
@pytest.mark.parametrize("block,shape", [(8, (40, 56)), (16, (90, 131)), (16, (64, 64)), (10, (61, 47))])
def test_match_per_block_regions(search, block, shape):
    """The per-block extension of Steps 4-5: own vectors, merge of equal vectors only (fast and generic kernels)."""
    g = rng(block + shape[1])
    H, W = shape
    prev, cur = two_motion_pair(g, H, W)
    smooth = np.clip(prev.astype(np.int32) + g.integers(-6, 7, size=prev.shape), 0, 255).astype(np.uint8)
    check_pairs([(prev, cur), (prev, prev), (prev, smooth), (cur, prev)], block, 4, search,
                region_mode=B.DC_REGIONS_PER_BLOCK)
    check_pairs([(prev, cur)], block, 4, search, skip_k=2, region_mode=B.DC_REGIONS_PER_BLOCK)


def test_match_per_block_streams_and_full_hd():
    w = configs.WORKLOADS[4]()
    sb = w.streams(1, 4)
    check_pairs([(sb.frame(i - 1)[0], sb.frame(i)[0]) for i in (1, 2, 3)], 16, 24, B.DC_SEARCH_DIAMOND,
                region_mode=B.DC_REGIONS_PER_BLOCK)
    w = configs.WORKLOADS[5]()
    sb = w.streams(2, 3)
    check_pairs([(sb.frame(1, s), sb.frame(2, s)) for s in range(2)], 16, 32, B.DC_SEARCH_DIAMOND,
                region_mode=B.DC_REGIONS_PER_BLOCK)


@pytest.mark.parametrize("widx", [2, 3, 4])
def test_infer_per_block_regions(widx):
    U.run_stream_parity(configs.WORKLOADS[widx](), 1, list(range(4)), region_mode=B.DC_REGIONS_PER_BLOCK)


@pytest.mark.parametrize("widx,frames", [(2, 6), (3, 5), (5, 3)])
def test_infer_with_cached_pooling(widx, frames):
    """Reuse in max-pooling layers (the extension Section 5 mentions): maps, rectangles and per-layer reuse ratios
    of the pooling layers against the oracle with the same switch."""
    w = configs.WORKLOADS[widx]()
    U.run_stream_parity(w, 2 if widx == 5 else 1, list(range(frames)), cache_pool=True)


def test_cached_pooling_reuses_pixels():
    w = configs.WORKLOADS[2]()
    sb = w.streams(1, 3)
    dc = DeepCache.from_workload(w, cache_pool=True)
    try:
        for i in range(3):
            out, stats = dc.infer_frame(sb.frame(i), want_stats=True)
        pools = [i for i, l in enumerate(w.layers) if l["kind"] == orc.KIND_MAXPOOL]
        assert pools and all(stats[0].reuse_ratio[i] > 0.2 for i in pools)
    finally:
        dc.close()


@pytest.mark.parametrize("dtype", [configs.DTYPE_FP32, configs.DTYPE_BF16])
def test_infer_graph_with_every_layer_kind(dtype):
    """Convolution, LRN, pooling, two branches joined by a concat and a fully-connected head (all rows of Table 2),
    every layer's map and rectangles against the oracle over a refresh, cached frames and the next refresh."""
    w = configs.WORKLOADS[2]()
    w.layers = nets.inception_lrn_net(80, 96)
    w.width, w.height, w.dtype, w.expire_n = 96, 80, dtype, 3
    crop = w.make_streams
    w.make_streams = lambda s, f, first=0: _cropped(crop(s, f, first), 80, 96)
    U.run_stream_parity(w, 2, list(range(5)))
    U.run_stream_parity(w, 1, list(range(3)), cache_pool=True, region_mode=B.DC_REGIONS_PER_BLOCK)


class _cropped:
    """A stream batch cut to the top-left h x w pixels of every frame."""

    def __init__(self, batch, h, w):
        self.batch, self.h, self.w = batch, h, w

    def frame(self, i, s=None):
        f = self.batch.frame(i) if s is None else self.batch.frame(i, s)
        return np.ascontiguousarray(f[..., :self.h, :self.w, :])


@pytest.mark.parametrize("k", [2, 3])
def test_match_k_skip(k):
    """Section 4's k-skip: Step 2 on every k-th block row and column only (16-px fast path and generic path)."""
    w = configs.WORKLOADS[2]()
    sb = w.streams(1, 4)
    pairs = [(sb.frame(i - 1)[0], sb.frame(i)[0]) for i in (1, 2, 3)]
    check_pairs(pairs, 16, 16, B.DC_SEARCH_DIAMOND, skip_k=k)
    check_pairs(pairs, 10, 6, B.DC_SEARCH_DIAMOND, skip_k=k)
    check_pairs([(p[:96, :96], c[:96, :96]) for p, c in pairs], 8, 3, B.DC_SEARCH_EXHAUSTIVE, skip_k=k)


def test_infer_with_k_skip():
    U.run_stream_parity(configs.WORKLOADS[3](), 1, list(range(5)), skip_k=2)


def test_match_needs_a_key():
    dc = matcher_only(32, 32, 1, 8, 4, B.DC_SEARCH_DIAMOND)
    try:
        with pytest.raises(B.DeepCacheError) as e:
            dc.match_blocks(np.zeros((32, 32, 3), np.uint8))
        assert e.value.status == B.DC_ERR_STATE
    finally:
        dc.close()


# ------------------------------------------------------------------ dc_propagate_regions
def random_regions(g, n, W, H, max_shift=9):
    out = np.zeros(n, orc.REGION_DTYPE)
    for i in range(n):
        w, h = int(g.integers(1, W // 2)), int(g.integers(1, H // 2))
        x, y = int(g.integers(0, W - w + 1)), int(g.integers(0, H - h + 1))
        sx = int(np.clip(x + g.integers(-max_shift, max_shift + 1), 0, W - w))
        sy = int(np.clip(y + g.integers(-max_shift, max_shift + 1), 0, H - h))
        out[i] = (x, y, w, h, sx, sy)
    return out


def check_propagation(layers, W, H, n_streams, executable=True):
    g = rng(len(layers))
    if executable:
        ws, bs = nets.random_weights(layers, 2)
    else:
        ws, bs = [None] * len(layers), [None] * len(layers)
    dc = DeepCache(W, H, layers, ws, bs, n_streams=n_streams, block=16, search_range=8, dtype=B.DC_BF16)
    try:
        regs = torch.zeros((n_streams, dc.max_regions, 6), dtype=torch.int32)
        counts, per_stream = [], []
        for s in range(n_streams):
            n = int(g.integers(0, min(dc.max_regions, 40) + 1)) if s else min(dc.max_regions, 37)
            r = random_regions(g, n, W, H)
            per_stream.append(r)
            counts.append(n)
            if n:
                regs[s, :n] = torch.from_numpy(np.ascontiguousarray(r).view(np.int32).reshape(n, 6))
        out, n_out = dc.propagate_regions(regs.cuda(), torch.tensor(counts, dtype=torch.int32).cuda())
        for s in range(n_streams):
            want = orc.propagate(layers, (H, W), per_stream[s])
            for li in range(len(layers)):
                U.assert_regions_equal(U.regions_np(out[li, s, :counts[s]]), want[li], f"layer {li} stream {s}")
                assert int(n_out[li, s]) == counts[s]
                assert not out[li, s, counts[s]:].any()
    finally:
        dc.close()


@pytest.mark.parametrize("net,W,H", [("small", 227, 227), ("alexnet", 227, 227), ("resnet", 224, 224), ("vgg", 1920, 1080)])
def test_propagate_networks(net, W, H):
    layers = {"small": lambda: nets.small_cnn(H, W), "alexnet": lambda: nets.alexnet_trunk(H, W),
              "resnet": lambda: nets.resnet50_trunk(H, W), "vgg": lambda: nets.vgg16_trunk(224, 224, H, W)}[net]()
    check_propagation(layers, W, H, 3)


def test_propagate_table2_rows():
    """Layer kinds that only region propagation knows (LRN, concat, fully connected)."""
    b = nets.NetBuilder(96, 96)
    c1 = b.conv(-1, 16, 11, 2, 5)
    b.layers.append(dict(kind=B.DC_RELU, kh=1, kw=1, sh=1, sw=1, ph=0, pw=0, cin=16, cout=16, relu=0, in0=c1, in1=-1, out_h=48, out_w=48))
    b.layers.append(dict(kind=B.DC_LRN, kh=5, kw=5, sh=1, sw=1, ph=2, pw=2, cin=16, cout=16, relu=0, in0=1, in1=-1, out_h=48, out_w=48))
    p = b.maxpool(2, 3, 2, 1)
    q = b.conv(2, 16, 3, 2, 1)
    b.layers.append(dict(kind=B.DC_CONCAT, kh=1, kw=1, sh=1, sw=1, ph=0, pw=0, cin=16, cout=32, relu=0, in0=p, in1=q, out_h=24, out_w=24))
    b.layers.append(dict(kind=B.DC_FC, kh=1, kw=1, sh=1, sw=1, ph=0, pw=0, cin=32, cout=10, relu=0, in0=5, in1=-1, out_h=1, out_w=1))
    check_propagation(b.layers, 96, 96, 2, executable=False)


# ------------------------------------------------------------------ dc_conv_partial
@pytest.mark.parametrize("dtype", [B.DC_FP32, B.DC_BF16])
@pytest.mark.parametrize("hi,wi,cin,cout,k,s,p,relu", [
    (37, 45, 3, 16, 3, 1, 1, 1), (64, 64, 32, 64, 3, 1, 1, 1), (227, 227, 3, 96, 11, 4, 0, 1),
    (27, 27, 96, 256, 5, 1, 2, 1), (56, 56, 64, 128, 1, 2, 0, 0), (30, 33, 16, 24, 3, 2, 1, 0),
    (14, 14, 256, 512, 3, 1, 1, 1), (224, 224, 3, 64, 7, 2, 3, 1), (40, 52, 3, 64, 3, 1, 1, 1),
    (33, 35, 3, 32, 5, 1, 2, 0), (28, 28, 32, 96, 3, 1, 1, 1), (20, 24, 16, 64, 1, 1, 0, 1),
    (28, 28, 64, 64, 3, 2, 1, 1), (31, 29, 128, 64, 3, 2, 1, 0), (40, 40, 32, 32, 5, 3, 2, 1)])
def test_conv_partial(dtype, hi, wi, cin, cout, k, s, p, relu):
    g = rng(hi + cin + k)
    bf16 = dtype == B.DC_BF16
    quant = orc.QUANT_BF16 if bf16 else orc.QUANT_NONE
    S = 2
    b = nets.NetBuilder(hi, wi, cin)
    b.conv(-1, cout, k, s, p, relu)
    L = b.layers[0]
    wts = g.normal(0, np.sqrt(2.0 / (k * k * cin)), size=(cout, k, k, cin)).astype(np.float32)
    bias = g.normal(0, 0.1, size=cout).astype(np.float32)
    layers = [dict(L)]
    x = g.normal(size=(S, hi, wi, cin))
    prev = g.normal(size=(S, L["out_h"], L["out_w"], cout))
    # inputs exactly representable in the map's element type, so copies can be compared bit for bit
    x, prev = x.astype(np.float32).astype(np.float64), prev.astype(np.float32).astype(np.float64)
    xq = np.stack([orc.quant_array(v, quant) for v in x])
    pq = np.stack([orc.quant_array(v, quant) for v in prev])
    tdt = torch.bfloat16 if bf16 else torch.float32
    # the library validates cin against the frame's 3 channels for in0 = -1, so give the conv a
    # producer with the right shape when cin != 3: a 1x1 conv from the frame stands in
    if cin == 3:
        net, li, fh, fw = layers, 0, hi, wi
        ws, bs = [wts], [bias]
    else:
        nb = nets.NetBuilder(hi, wi)
        a = nb.conv(-1, cin, 1, 1, 0)
        nb.conv(a, cout, k, s, p, relu)
        net, li, fh, fw = nb.layers, 1, hi, wi
        ws = [np.zeros((cin, 1, 1, 3), np.float32), wts]
        bs = [np.zeros(cin, np.float32), bias]
    dc = DeepCache(fw, fh, net, ws, bs, n_streams=S, block=16, search_range=4, dtype=dtype, max_regions=8)
    try:
        regs = torch.zeros((S, dc.max_regions, 6), dtype=torch.int32)
        per_stream, counts = [], []
        for s_ in range(S):
            n = min(dc.max_regions, 6)
            # disjoint rectangles: split the output into a grid of cells, one rectangle inside each
            r = np.zeros(n, orc.REGION_DTYPE)
            cw, ch = L["out_w"] // 3, L["out_h"] // 2
            for i in range(n):
                cx, cy = (i % 3) * cw, (i // 3) * ch
                w_ = int(g.integers(1, cw + 1)); h_ = int(g.integers(1, ch + 1))
                x0 = cx + int(g.integers(0, cw - w_ + 1)); y0 = cy + int(g.integers(0, ch - h_ + 1))
                sx = int(g.integers(0, L["out_w"] - w_ + 1)); sy = int(g.integers(0, L["out_h"] - h_ + 1))
                r[i] = (x0, y0, w_, h_, sx, sy)
            if s_ == 1:
                r[2] = (0, 0, 0, 0, 0, 0)          # a vanished slot
            per_stream.append(r); counts.append(n)
            regs[s_, :n] = torch.from_numpy(np.ascontiguousarray(r).view(np.int32).reshape(n, 6))
        xin = torch.from_numpy(xq).to(tdt).cuda()
        pin = torch.from_numpy(pq).to(tdt).cuda()
        full = dc.conv_partial(li, xin)
        part = dc.conv_partial(li, xin, pin, regs.cuda(), torch.tensor(counts, dtype=torch.int32).cuda())
        wq = orc.quant_array(wts, quant)
        for s_ in range(S):
            want_full, _ = orc.conv_reuse(xq[s_], L, wq, bias, quant)
            want, reused = orc.conv_reuse(xq[s_], L, wq, bias, quant, pq[s_], per_stream[s_])
            U.assert_map_close(full[s_], want_full, bf16, "full")
            U.assert_map_close(part[s_], want, bf16, "partial")
            if bf16:
                U.assert_map_close_per_element(full[s_], want_full, "full, per element")
            m = reused.astype(bool)
            got = part[s_].float().cpu().numpy().astype(np.float64)
            assert m.any() and np.array_equal(got[m], want[m]), "reused pixels must be bit-equal copies of the cached map"
        assert dc.status() == B.DC_OK
    finally:
        dc.close()


def test_conv_partial_ignores_rectangles_outside_the_map():
    """A caller's rectangle that leaves the map on either side, or a count beyond max_regions, must not become an
    out-of-bounds access: such rectangles are not reused (their pixels are convolved) and the status word says so."""
    g = rng(77)
    hi, wi, cout = 37, 45, 16
    b = nets.NetBuilder(hi, wi, 3)
    b.conv(-1, cout, 3, 1, 1, 1)
    L = b.layers[0]
    wts = g.normal(0, 0.2, size=(cout, 3, 3, 3)).astype(np.float32)
    bias = g.normal(0, 0.1, size=cout).astype(np.float32)
    x = g.normal(size=(1, hi, wi, 3)).astype(np.float32).astype(np.float64)
    prev = g.normal(size=(1, hi, wi, cout)).astype(np.float32).astype(np.float64)
    dc = DeepCache(wi, hi, [dict(L)], [wts], [bias], n_streams=1, block=16, search_range=4, dtype=B.DC_FP32, max_regions=8)
    try:
        good = (4, 5, 10, 9, 7, 2)
        bad = [(30, 3, 10, 6, 40, 3),            # cached side leaves the map on the right
               (2, 30, 5, 6, 2, -1),             # cached side starts above the map
               (-3, 20, 8, 4, 0, 20),            # current side starts left of the map
               (20, 20, 100, 4, 0, 0),           # wider than the map
               (10, 25, 2 ** 30, 2 ** 30, 5, 5),  # sizes that would overflow a sum
               (12, 12, -4, 3, 1, 1)]            # negative width: an empty slot, not an error
        regs = torch.zeros((1, dc.max_regions, 6), dtype=torch.int32)
        for i, r in enumerate([good] + bad):
            regs[0, i] = torch.tensor(r, dtype=torch.int32)
        xin, pin = torch.from_numpy(x).float().cuda(), torch.from_numpy(prev).float().cuda()
        # a count far beyond the table: cut to max_regions (the eighth slot is all zeros)
        part = dc.conv_partial(0, xin, pin, regs.cuda(), torch.tensor([1000], dtype=torch.int32).cuda())
        only_good = np.zeros(1, orc.REGION_DTYPE); only_good[0] = good
        want, reused = orc.conv_reuse(x[0], L, wts, bias, orc.QUANT_NONE, prev[0], only_good)
        U.assert_map_close(part[0], want, False, "bad rectangles ignored")
        m = reused.astype(bool)
        assert np.array_equal(part[0].cpu().numpy().astype(np.float64)[m], want[m])
        assert dc.status() == B.DC_ERR_ARG
        dc.reset()
        assert dc.status() == B.DC_OK
    finally:
        dc.close()


@pytest.mark.parametrize("scheme", [1, 2, 3, 4, 5, 6, 7, 8, 9])
def test_conv_schemes_forced(scheme, monkeypatch):
    """Every operand scheme of the tensor-core convolution (tap by tap, patch, column slabs; one or two tiles per
    item; column slabs on CTA pairs; tap by tap on flat tiles) on layers it can take: VGG-shaped 3x3 layers, a 5x5 layer and odd map sizes,
    through cached frames."""
    monkeypatch.setenv("DC_CONV_SCHEME", str(scheme))
    b = nets.NetBuilder(45, 53)
    x = b.conv(-1, 64, 3, 1, 1)
    x = b.conv(x, 64, 3, 1, 1)
    x = b.conv(x, 128, 5, 1, 2)
    x = b.maxpool(x, 2, 2)
    x = b.conv(x, 256, 3, 1, 1)
    b.conv(x, 256, 3, 1, 1, relu=0)
    w = configs.small_cnn_stream()
    w.layers, w.dtype, w.width, w.height = b.layers, configs.DTYPE_BF16, 53, 45
    inner = w.make_streams
    w.make_streams = lambda s, f, first=0: _cropped(inner(s, f), 45, 53)
    U.run_stream_parity(w, 2, [0, 1, 2])


# ------------------------------------------------------------------ dc_infer_frame
def test_infer_workload_1():
    U.run_stream_parity(configs.WORKLOADS[1](), 1, [0, 1])


def test_infer_workload_2_through_an_expiry():
    U.run_stream_parity(configs.WORKLOADS[2](), 1, list(range(12)))


def test_infer_workload_3_alexnet_bf16():
    U.run_stream_parity(configs.WORKLOADS[3](), 1, list(range(12)))


@pytest.mark.parametrize("dtype", [configs.DTYPE_FP32, configs.DTYPE_BF16])
def test_infer_alexnet_with_grouped_convolutions(dtype):
    """The AlexNet trunk with two channel groups in its second, fourth and fifth convolutions: every layer's
    rectangles, reuse ratios and maps against the oracle, cached frames included."""
    w = configs.alexnet_stream(grouped=True, dtype=dtype)
    U.run_stream_parity(w, 1, list(range(4)))
    # in bfloat16 every convolution, the grouped ones included, runs on the tensor-core kernels (one launch per group)
    dc = DeepCache.from_workload(w, n_streams=1)
    try:
        schemes = [B.dc_cache_layer_conv_scheme(dc.handle, i) for i, l in enumerate(w.layers) if l["kind"] == 0]
        assert len(schemes) == 5 and any(l.get("groups", 1) > 1 for l in w.layers)
        assert all(v >= 1 for v in schemes) if dtype == configs.DTYPE_BF16 else all(v == 0 for v in schemes)
    finally:
        dc.close()


def test_infer_workload_4_resnet50_bf16():
    U.run_stream_parity(configs.WORKLOADS[4](), 1, list(range(4)))


@pytest.mark.parametrize("wid,frames", [(3, [0, 1, 2]), (4, [0, 1])])
def test_infer_small_map_trunks_three_streams(wid, frames):
    """The AlexNet and ResNet-50 trunks with three streams in one cache: tiles of their small maps may hold pixels of
    two streams (flat tiles), and their strided first layers run on the space-to-depth copy; every layer's map of
    every stream against the oracle."""
    U.run_stream_parity(configs.WORKLOADS[wid](), 3, frames)


def test_infer_workload_5_two_streams():
    """Full-HD matching, area resize to 224x224, VGG-16 trunk; 2 of the 32 streams, frames 0-2."""
    U.run_stream_parity(configs.WORKLOADS[5](), 2, [0, 1, 2])


def test_infer_workload_5_full_batch_sampled_streams():
    """The benchmark's own configuration: all 32 full-HD streams in one cache, the loop bench.py times
    (dc_infer_frame(t), then dc_lookahead_frame(t + 1)), frames 0-3.  The oracle follows three of the streams
    (first, one in the middle, last): motion vector, counts, frame rectangles and the final map of every frame."""
    w = configs.WORKLOADS[5]()
    S, n_frames, sample = w.n_streams, 4, (0, 13, w.n_streams - 1)
    bf16 = w.dtype == configs.DTYPE_BF16
    sb = w.streams(S, n_frames)
    frames = [torch.from_numpy(np.ascontiguousarray(sb.frame(i))).cuda() for i in range(n_frames)]
    oracles = dict(zip(sample, U.make_oracles(w, len(sample))))
    dc = DeepCache.from_workload(w, n_streams=S)
    try:
        pitch = w.width * 3
        for i in range(n_frames):
            out, st = dc.infer_frame(frames[i], want_stats=True)
            out = out.clone()
            regs0, _ = dc.layer_regions(-1)
            regs0 = regs0.clone()
            if i + 1 < n_frames:
                B.dc_lookahead_frame(dc.handle, frames[i + 1], pitch)
            for s in sample:
                o = oracles[s].infer_frame(sb.frame(i, s))
                what = f"frame {i} stream {s} of {S}"
                assert bool(st[s].refreshed) == o["refreshed"], what
                if not o["refreshed"]:
                    m = o["match"]
                    assert (st[s].mvx, st[s].mvy, st[s].k_passed) == (m["M"][0], m["M"][1], m["K"]), what
                    assert st[s].n_matched == int(m["matched"].sum()) and st[s].n_regions == len(m["regions"]), what
                    U.assert_regions_equal(U.regions_np(regs0[s, :len(m["regions"])]), m["regions"], what + " frame rectangles")
                U.assert_map_close(out[s], o["out"], bf16, what + " output")
        assert dc.status() == B.DC_OK
    finally:
        dc.close()


def test_infer_identical_frames_and_reset():
    w = configs.WORKLOADS[2]()
    f = w.streams(1, 1).frame(0)
    dc = DeepCache.from_workload(w)
    try:
        a = dc.infer_frame(f).clone()
        b, st = dc.infer_frame(f, want_stats=True)
        assert not st[0].refreshed and (st[0].mvx, st[0].mvy) == (0, 0) and st[0].n_regions == 1
        assert torch.equal(a, b)                     # everything reusable was copied, the rest recomputed identically
        dc.reset()
        c, st = dc.infer_frame(f, want_stats=True)
        assert st[0].refreshed and torch.equal(a, c)
    finally:
        dc.close()


def test_infer_host_buffers_with_and_without_prefetch():
    """dc_infer_frame_host (host frames in, last map out) with the next frame prefetched, without, and with a
    prefetch that is then not used: all equal dc_infer_frame on device buffers, bit for bit."""
    w = configs.WORKLOADS[2]()
    sb = w.streams(1, 6)
    frames = [torch.from_numpy(np.ascontiguousarray(sb.frame(i))).pin_memory() for i in range(6)]
    ref = DeepCache.from_workload(w)
    dc = DeepCache.from_workload(w)
    try:
        pitch = w.width * 3
        out_host = torch.empty(ref.out_shape(-1), dtype=torch.float32).pin_memory()
        B.dc_prefetch_frame_host(dc.handle, frames[0].data_ptr(), pitch)
        for i in range(6):
            want = ref.infer_frame(frames[i].cuda())
            if i in (0, 1, 3):                        # the usual loop: prefetch the next frame, then compute this one
                B.dc_prefetch_frame_host(dc.handle, frames[i + 1].data_ptr(), pitch)
            B.dc_infer_frame_host(dc.handle, frames[i].data_ptr(), pitch, out_host.data_ptr())
            assert torch.equal(out_host, want.cpu()), f"frame {i}"
        # a third pending prefetch is refused
        B.dc_prefetch_frame_host(dc.handle, frames[0].data_ptr(), pitch)
        B.dc_prefetch_frame_host(dc.handle, frames[1].data_ptr(), pitch)
        with pytest.raises(B.DeepCacheError) as e:
            B.dc_prefetch_frame_host(dc.handle, frames[2].data_ptr(), pitch)
        assert e.value.status == B.DC_ERR_STATE
        assert dc.status() == B.DC_OK
    finally:
        ref.close(); dc.close()


def test_region_overflow_sets_the_status_word():
    """More rectangles than max_regions: the extra ones are dropped and the device status word says so."""
    prev = rng(2).integers(0, 256, size=(64, 64, 3), dtype=np.uint8)
    cur = prev.copy()
    cur[::16, :] = 255 - cur[::16, :]                 # ruin every other 8-px block row: matched rows alternate
    cur[:, 24:32] = 255 - cur[:, 24:32]               # and one block column: two runs per matched row
    layers = nets.single_conv(64, 64)
    ws, bs = nets.random_weights(layers, 1)
    want = orc.match_blocks(cur, prev, 8, 2, orc.SEARCH_DS, 20.0)
    assert len(want["regions"]) > 2
    dc = DeepCache(64, 64, layers, ws, bs, block=8, search_range=2, max_regions=2)
    try:
        dc.set_key(prev)
        got = dc.match_blocks(cur)
        assert int(got["n_regions"][0]) == 2
        U.assert_regions_equal(U.regions_np(got["regions"][0, :2]), want["regions"][:2], "kept rectangles")
        assert dc.status() == B.DC_ERR_OVERFLOW
        dc.reset()
        assert dc.status() == B.DC_OK
    finally:
        dc.close()


@pytest.mark.parametrize("scheme", [5, 7])
@pytest.mark.parametrize("hi,wi,cin,cout,k,p", [(14, 14, 256, 512, 3, 1), (28, 28, 128, 256, 3, 1), (17, 23, 64, 128, 5, 2), (9, 40, 128, 256, 1, 0)])
def test_conv_wide_layers_on_cta_pairs(scheme, hi, wi, cin, cout, k, p, monkeypatch):
    """The wide layers (128 - 512 output channels) forced onto the CTA-pair kernel (7), and onto the single-CTA column-slab
    kernel (5) for comparison: full convolution and partial convolution with an odd number of dirty tiles."""
    monkeypatch.setenv("DC_CONV_SCHEME", str(scheme))
    _one_layer_full_and_partial(hi, wi, cin, cout, k, 1, p, 3, scheme)


@pytest.mark.parametrize("scheme", [8, 9])
@pytest.mark.parametrize("hi,wi,cin,cout,k,st,p,S", [
    (7, 7, 128, 256, 3, 1, 1, 5),        # 7 pieces per stream: every tile holds pieces of two or three streams
    (14, 14, 256, 512, 3, 1, 1, 3),      # two pieces per row
    (13, 13, 64, 96, 3, 1, 1, 4),        # a cut last piece in every row; 32-channel blocks
    (27, 27, 32, 64, 5, 2, 2, 3),        # a strided layer (14 x 14 output), 64-byte operand rows
    (9, 40, 128, 256, 1, 1, 0, 3),       # 1 x 1
    (3, 5, 64, 64, 3, 1, 1, 1),          # one tile, mostly absent
])
def test_conv_flat_tiles_across_rows_and_streams(scheme, hi, wi, cin, cout, k, st, p, S, monkeypatch):
    """Small maps on tiles made of 16 row pieces of 8 pixels that run on across rows and streams (scheme 8; 9 with two
    tiles per item): the reuse bitmap, the dirty list and the copies then follow that numbering too."""
    monkeypatch.setenv("DC_CONV_SCHEME", str(scheme))
    _one_layer_full_and_partial(hi, wi, cin, cout, k, st, p, S, scheme)


def _one_layer_full_and_partial(hi, wi, cin, cout, k, st, p, S, scheme):
    g = rng(hi * 7 + cout)
    nb = nets.NetBuilder(hi, wi)
    a = nb.conv(-1, cin, 1, 1, 0)
    nb.conv(a, cout, k, st, p, 1)
    L = nb.layers[1]
    wts = g.normal(0, np.sqrt(2.0 / (k * k * cin)), size=(cout, k, k, cin)).astype(np.float32)
    bias = g.normal(0, 0.1, size=cout).astype(np.float32)
    ws = [np.zeros((cin, 1, 1, 3), np.float32), wts]
    bs = [np.zeros(cin, np.float32), bias]
    xq = np.stack([orc.quant_array(g.normal(size=(hi, wi, cin)), orc.QUANT_BF16) for _ in range(S)])
    pq = np.stack([orc.quant_array(g.normal(size=(L["out_h"], L["out_w"], cout)), orc.QUANT_BF16) for _ in range(S)])
    dc = DeepCache(wi, hi, nb.layers, ws, bs, n_streams=S, block=16, search_range=4, dtype=B.DC_BF16, max_regions=4)
    try:
        if scheme >= 8:
            assert B.dc_cache_layer_conv_scheme(dc.handle, 1) == scheme
        xin = torch.from_numpy(xq).to(torch.bfloat16).cuda()
        pin = torch.from_numpy(pq).to(torch.bfloat16).cuda()
        full = dc.conv_partial(1, xin)
        # one rectangle that covers the whole map of stream 1 (its tiles are clean: the dirty count becomes odd for
        # most shapes) and a small one in stream 0
        regs = torch.zeros((S, dc.max_regions, 6), dtype=torch.int32)
        counts = torch.zeros(S, dtype=torch.int32)
        ow, oh = L["out_w"], L["out_h"]
        regs[0, 0] = torch.tensor([1, 2, min(5, ow - 2), min(4, oh - 2), 2, 1] if oh >= 4 else [1, 1, ow - 1, oh - 1, 0, 0], dtype=torch.int32)
        counts[0] = 1
        if S > 1:
            regs[1, 0] = torch.tensor([0, 0, ow, oh, 0, 0], dtype=torch.int32)
            counts[1] = 1
        part = dc.conv_partial(1, xin, pin, regs.cuda(), counts.cuda())
        wq = orc.quant_array(wts, orc.QUANT_BF16)
        for s_ in range(S):
            r = np.zeros(1, orc.REGION_DTYPE)
            r[0] = tuple(int(v) for v in regs[s_, 0])
            want_full, _ = orc.conv_reuse(xq[s_], L, wq, bias, orc.QUANT_BF16)
            want, reused = orc.conv_reuse(xq[s_], L, wq, bias, orc.QUANT_BF16, pq[s_], r[:int(counts[s_])])
            U.assert_map_close(full[s_], want_full, True, f"full, stream {s_}")
            U.assert_map_close_per_element(full[s_], want_full, f"full, per element, stream {s_}")
            U.assert_map_close(part[s_], want, True, f"partial, stream {s_}")
            m = reused.astype(bool)
            got = part[s_].float().cpu().numpy().astype(np.float64)
            assert np.array_equal(got[m], want[m])
        assert dc.status() == B.DC_OK
    finally:
        dc.close()


@pytest.mark.parametrize("hi,wi,cout,k,st,p,S", [
    (59, 63, 96, 11, 4, 0, 3),       # AlexNet's first layer: 4 x 4 blocks of 3 channels = 48 -> 64 channels, 3 x 3 taps
    (45, 53, 64, 7, 2, 3, 2),        # ResNet's stem: 2 x 2 blocks = 12 -> 16 channels, 4 x 4 taps, three zero rows in front
    (37, 41, 32, 5, 2, 2, 2),
    (30, 34, 64, 3, 2, 1, 1),
    (40, 43, 32, 7, 3, 2, 2),        # 3 x 3 blocks = 27 -> 32 channels
    (33, 35, 64, 11, 4, 2, 2),       # padding that is not a multiple of the stride
])
def test_conv_strided_first_layers_as_space_to_depth(hi, wi, cout, k, st, p, S):
    """Strided convolutions on RGB run as stride-1 convolutions over a space-to-depth copy of their input: full and
    partial convolution against the oracle's strided one."""
    g = rng(hi * 3 + k)
    nb = nets.NetBuilder(hi, wi)
    nb.conv(-1, cout, k, st, p, 1)
    L = nb.layers[0]
    oh, ow = L["out_h"], L["out_w"]
    wts = g.normal(0, np.sqrt(2.0 / (k * k * 3)), size=(cout, k, k, 3)).astype(np.float32)
    bias = g.normal(0, 0.1, size=cout).astype(np.float32)
    xq = np.stack([orc.quant_array(g.uniform(0, 1, size=(hi, wi, 3)), orc.QUANT_BF16) for _ in range(S)])
    pq = np.stack([orc.quant_array(g.normal(size=(oh, ow, cout)), orc.QUANT_BF16) for _ in range(S)])
    dc = DeepCache(wi, hi, nb.layers, [wts], [bias], n_streams=S, block=16, search_range=4, dtype=B.DC_BF16, max_regions=4)
    try:
        assert B.dc_cache_layer_conv_scheme(dc.handle, 0) >= 1          # a tensor-core scheme
        xin = torch.from_numpy(xq).to(torch.bfloat16).cuda()
        pin = torch.from_numpy(pq).to(torch.bfloat16).cuda()
        full = dc.conv_partial(0, xin)
        regs = torch.zeros((S, dc.max_regions, 6), dtype=torch.int32)
        counts = torch.zeros(S, dtype=torch.int32)
        regs[0, 0] = torch.tensor([1, 2, min(5, ow - 2), min(4, oh - 3), 2, 1], dtype=torch.int32)
        counts[0] = 1
        part = dc.conv_partial(0, xin, pin, regs.cuda(), counts.cuda())
        wq = orc.quant_array(wts, orc.QUANT_BF16)
        for s_ in range(S):
            r = np.zeros(1, orc.REGION_DTYPE)
            r[0] = tuple(int(v) for v in regs[s_, 0])
            want_full, _ = orc.conv_reuse(xq[s_], L, wq, bias, orc.QUANT_BF16)
            want, reused = orc.conv_reuse(xq[s_], L, wq, bias, orc.QUANT_BF16, pq[s_], r[:int(counts[s_])])
            U.assert_map_close(full[s_], want_full, True, f"full, stream {s_}")
            U.assert_map_close_per_element(full[s_], want_full, f"full, per element, stream {s_}")
            U.assert_map_close(part[s_], want, True, f"partial, stream {s_}")
            m = reused.astype(bool)
            got = part[s_].float().cpu().numpy().astype(np.float64)
            assert np.array_equal(got[m], want[m])
        assert dc.status() == B.DC_OK
    finally:
        dc.close()


@pytest.mark.parametrize("cin,k", [(64, 3), (32, 1), (3, 3), (128, 7)])      # column-slab / patch kernels, tap-by-tap kernel, few-channel kernel, CTA pairs
def test_bounded_device_waits_run_out_and_the_cache_stays_usable(cin, k, monkeypatch):
    """Failure detection without a fault: one convolution launch is armed so that its producer issues no copy.  The
    other roles' waits then run out after a few milliseconds instead of spinning for ever: the kernel returns, the
    status word reads DC_ERR_TIMEOUT, tensor memory is free again, and the next launch on the same cache is correct."""
    import ctypes
    g = rng(90 + cin)
    hi = wi = 40
    cout = 64
    if k == 7:                                                     # stands for: a 3x3 layer of 128 -> 256 channels forced onto CTA pairs
        k, cout = 3, 256
        monkeypatch.setenv("DC_CONV_SCHEME", "7")
    nb = nets.NetBuilder(hi, wi)
    if cin == 3:
        nb.conv(-1, cout, k, 1, k // 2, 1)
        li = 0
        ws = [g.normal(0, 0.2, size=(cout, k, k, 3)).astype(np.float32)]
        bs = [g.normal(0, 0.1, size=cout).astype(np.float32)]
    else:
        a = nb.conv(-1, cin, 1, 1, 0)
        nb.conv(a, cout, k, 1, k // 2, 1)
        li = 1
        ws = [np.zeros((cin, 1, 1, 3), np.float32), g.normal(0, 0.1, size=(cout, k, k, cin)).astype(np.float32)]
        bs = [np.zeros(cin, np.float32), g.normal(0, 0.1, size=cout).astype(np.float32)]
    L = nb.layers[li]
    x = orc.quant_array(g.normal(size=(hi, wi, cin)), orc.QUANT_BF16)
    want, _ = orc.conv_reuse(x, L, orc.quant_array(ws[li], orc.QUANT_BF16), bs[li], orc.QUANT_BF16)
    dc = DeepCache(wi, hi, nb.layers, ws, bs, n_streams=1, block=16, search_range=4, dtype=B.DC_BF16)
    try:
        stall = B.load().dc_debug_stall_next_conv
        stall.restype = ctypes.c_int
        stall.argtypes = [ctypes.c_void_p, ctypes.c_int]
        xin = torch.from_numpy(x[None]).to(torch.bfloat16).cuda()
        U.assert_map_close(dc.conv_partial(li, xin)[0], want, True, "before")
        assert dc.status() == B.DC_OK
        assert stall(dc.handle, 5) == B.DC_OK
        dc.conv_partial(li, xin)                                   # returns normally; its output is not valid
        assert dc.status() == B.DC_ERR_TIMEOUT
        dc.reset()                                                 # clears the status word
        assert dc.status() == B.DC_OK
        U.assert_map_close(dc.conv_partial(li, xin)[0], want, True, "after")
        assert dc.status() == B.DC_OK
        assert stall(dc.handle, 0) == B.DC_ERR_ARG and stall(None, 5) == B.DC_ERR_ARG
    finally:
        dc.close()


def test_lookahead_gives_identical_results():
    """dc_lookahead_frame moves the matching of frame t+1 beside the inference of frame t; outputs, motion
    vectors and rectangles must not change.  Also: a lookahead for a frame that is then not used.
    One cache runs the sequence twice (plain, then with lookahead) so that both passes use the same kernels."""
    w = configs.WORKLOADS[3]()
    sb = w.streams(1, 13)
    frames = [torch.from_numpy(np.ascontiguousarray(sb.frame(i))).cuda() for i in range(13)]
    dc = DeepCache.from_workload(w)
    try:
        pitch = w.width * 3

        def run(lookahead):
            rec = []
            dc.reset()
            for i in range(12):
                out, st = dc.infer_frame(frames[i], want_stats=True)
                out = out.clone()
                if lookahead:
                    if i == 5:
                        B.dc_lookahead_frame(dc.handle, frames[0], pitch)        # announced, but frame 6 comes next
                    elif i != 7:
                        B.dc_lookahead_frame(dc.handle, frames[i + 1], pitch)    # crosses the expiry at frame 10
                regs, _ = dc.layer_regions(-1)
                key = (st[0].refreshed, st[0].mvx, st[0].mvy, st[0].k_passed, st[0].n_matched, st[0].n_regions)
                rec.append((out, key, regs[0, :st[0].n_regions].clone()))
            return rec

        plain, ahead = run(False), run(True)
        assert any(not k[0] and k[4] > 0 for _, k, _ in plain)
        for i, ((o0, k0, r0), (o1, k1, r1)) in enumerate(zip(plain, ahead)):
            assert k0 == k1, f"frame {i}: {k0} vs {k1}"
            if not k0[0]:
                assert torch.equal(r0, r1), f"frame {i} rectangles"
            assert torch.equal(o0, o1), f"frame {i} output"
        assert dc.status() == B.DC_OK
    finally:
        dc.close()
