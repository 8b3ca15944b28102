"""Pins for the oracle's layer arithmetic and its frame-by-frame cache semantics (Section 5)."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import deepcache_oracle as orc
from paper_1712_01670_b200.synth import configs, nets


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def conv_layer(hi, wi, cin, cout, k, s, p, relu=1):
    return dict(kind=orc.KIND_CONV, kh=k, kw=k, sh=s, sw=s, ph=p, pw=p, cin=cin, cout=cout, relu=relu,
                in0=-1, in1=-1, out_h=(hi + 2 * p - k) // s + 1, out_w=(wi + 2 * p - k) // s + 1)


@pytest.mark.parametrize("hi,wi,cin,cout,k,s,p,relu", [
    (13, 17, 3, 5, 3, 1, 1, 1), (23, 19, 4, 6, 11, 4, 0, 0), (16, 16, 8, 4, 5, 1, 2, 1),
    (15, 14, 6, 7, 1, 2, 0, 0), (20, 21, 3, 4, 7, 2, 3, 1), (9, 9, 2, 3, 3, 2, 1, 0)])
def test_conv_equals_torch_float64(hi, wi, cin, cout, k, s, p, relu):
    g = rng(hi * 100 + k)
    x = g.normal(size=(hi, wi, cin))
    w = g.normal(size=(cout, k, k, cin))
    b = g.normal(size=cout)
    L = conv_layer(hi, wi, cin, cout, k, s, p, relu)
    out, reused = orc.conv_reuse(x, L, w, b, orc.QUANT_NONE)
    ref = F.conv2d(torch.from_numpy(x).permute(2, 0, 1)[None], torch.from_numpy(w).permute(0, 3, 1, 2),
                   torch.from_numpy(b), stride=s, padding=p)
    if relu:
        ref = ref.clamp_min(0)
    ref = ref[0].permute(1, 2, 0).numpy()
    assert out.shape == ref.shape
    assert np.abs(out - ref).max() < 1e-12
    assert not reused.any()


@pytest.mark.parametrize("groups,cin,cout,k,s,p", [(2, 8, 12, 3, 1, 1), (4, 8, 8, 5, 2, 2), (3, 9, 6, 1, 1, 0), (2, 96, 64, 5, 1, 2)])
def test_grouped_conv_equals_torch_float64(groups, cin, cout, k, s, p):
    """Grouped convolution (the cited AlexNet's layers 2, 4, 5): library routine in float64, and the structural
    fact that an output channel does not depend on the input channels of another group."""
    g = rng(groups * 1000 + cin)
    hi, wi = 13, 17
    x = g.normal(size=(hi, wi, cin))
    w = g.normal(size=(cout, k, k, cin // groups))
    b = g.normal(size=cout)
    L = dict(conv_layer(hi, wi, cin, cout, k, s, p, 1), groups=groups)
    out, _ = orc.conv_reuse(x, L, w, b, orc.QUANT_NONE)
    ref = F.conv2d(torch.from_numpy(x).permute(2, 0, 1)[None], torch.from_numpy(w).permute(0, 3, 1, 2),
                   torch.from_numpy(b), stride=s, padding=p, groups=groups).clamp_min(0)[0].permute(1, 2, 0).numpy()
    assert np.abs(out - ref).max() < 1e-12
    x2 = x.copy()
    x2[..., :cin // groups] += 1.0                               # disturb group 0's inputs only
    out2, _ = orc.conv_reuse(x2, L, w, b, orc.QUANT_NONE)
    assert np.array_equal(out2[..., cout // groups:], out[..., cout // groups:])
    assert not np.array_equal(out2[..., :cout // groups], out[..., :cout // groups])
    # groups = 1 and a missing key are the ordinary convolution
    w1 = g.normal(size=(cout, k, k, cin))
    L1 = conv_layer(hi, wi, cin, cout, k, s, p, 0)
    a1, _ = orc.conv_reuse(x, dict(L1, groups=1), w1, b, orc.QUANT_NONE)
    L1.pop("groups", None)
    a0, _ = orc.conv_reuse(x, L1, w1, b, orc.QUANT_NONE)
    assert np.array_equal(a0, a1)


@pytest.mark.parametrize("k,s,p", [(2, 2, 0), (3, 2, 0), (3, 2, 1)])
def test_maxpool_equals_torch(k, s, p):
    g = rng(k + s)
    x = g.normal(size=(27, 23, 5))
    L = dict(kind=orc.KIND_MAXPOOL, kh=k, kw=k, sh=s, sw=s, ph=p, pw=p, cin=5, cout=5, relu=0, in0=-1, in1=-1,
             out_h=(27 + 2 * p - k) // s + 1, out_w=(23 + 2 * p - k) // s + 1)
    ref = F.max_pool2d(torch.from_numpy(x).permute(2, 0, 1)[None], k, s, p)[0].permute(1, 2, 0).numpy()
    assert np.array_equal(orc.maxpool(x, L), ref)


@pytest.mark.parametrize("h,w,ho,wo", [(108, 192, 22, 22), (50, 37, 7, 9), (64, 64, 64, 64), (30, 30, 15, 10)])
def test_resize_area_equals_adaptive_avg_pool(h, w, ho, wo):
    # adaptive average pooling uses the same spans: [floor(o n/no), ceil((o+1) n/no))
    f = rng(h).integers(0, 256, size=(h, w, 3), dtype=np.uint8)
    ref = F.adaptive_avg_pool2d(torch.from_numpy(f.astype(np.float64) / 255.0).permute(2, 0, 1)[None], (ho, wo))
    ref = ref[0].permute(1, 2, 0).numpy()
    assert np.abs(orc.resize_area(f, ho, wo, orc.QUANT_NONE) - ref).max() < 1e-14


def test_bf16_rounding_equals_torch():
    g = rng(1)
    v = np.concatenate([g.normal(size=2000) * 10.0 ** g.integers(-6, 6, size=2000),
                        [0.0, 1.0, -1.0, 1.00390625, 1.01171875, 255.5, 3.0e-5, 65504.0]])
    # exact ties: 1 + 2^-8 is halfway between 1 and 1 + 2^-7 -> even (1.0); 1 + 3*2^-8 -> 1 + 2^-6
    got = orc.quant_array(v, orc.QUANT_BF16)
    ref = torch.from_numpy(v).to(torch.float64).to(torch.bfloat16).to(torch.float64).numpy()
    # torch converts double -> float -> bf16; restrict to values where the float step is exact
    exact = v.astype(np.float32).astype(np.float64) == v
    assert np.array_equal(got[exact], ref[exact])
    assert orc.quant_array(np.array([1.00390625]), 1)[0] == 1.0
    assert orc.quant_array(np.array([1.01171875]), 1)[0] == 1.015625
    rel = np.abs(got - v) / np.maximum(np.abs(v), 1e-300)
    assert rel.max() <= 2.0 ** -8
    assert np.array_equal(orc.quant_array(got, 1), got)                 # idempotent


def test_input_map_is_pixel_over_255():
    f = np.arange(256, dtype=np.uint8).reshape(16, 16, 1).repeat(3, 2)
    assert np.array_equal(orc.input_map(f, orc.QUANT_NONE), f.astype(np.float64) / 255.0)
    q = orc.input_map(f, orc.QUANT_BF16)
    ref = torch.from_numpy(f.astype(np.float32) / np.float32(255.0)).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.abs(q - ref).max() <= 2.0 ** -8


def test_reused_pixels_are_cached_pixels_shifted():
    g = rng(6)
    hi, wi = 20, 24
    L = conv_layer(hi, wi, 3, 4, 3, 1, 1)
    x = g.normal(size=(hi, wi, 3))
    w = g.normal(size=(4, 3, 3, 3))
    b = g.normal(size=4)
    prev = g.normal(size=(hi, wi, 4))
    regions = np.zeros(3, orc.REGION_DTYPE)
    regions[0] = (2, 3, 6, 5, 4, 1)
    regions[1] = (0, 0, 0, 0, 0, 0)                      # vanished slot: ignored
    regions[2] = (12, 10, 10, 9, 11, 11)
    out, reused = orc.conv_reuse(x, L, w, b, orc.QUANT_NONE, prev, regions)
    full, _ = orc.conv_reuse(x, L, w, b, orc.QUANT_NONE)
    expect_mask = np.zeros((hi, wi), bool)
    for r in regions:
        expect_mask[r["y"]:r["y"] + r["h"], r["x"]:r["x"] + r["w"]] = True
        d = out[r["y"]:r["y"] + r["h"], r["x"]:r["x"] + r["w"]]
        s = prev[r["sy"]:r["sy"] + r["h"], r["sx"]:r["sx"] + r["w"]]
        assert np.array_equal(d, s)                      # bit-equal copies of the cached values
    assert np.array_equal(reused.astype(bool), expect_mask)
    assert np.array_equal(out[~expect_mask], full[~expect_mask])      # everything else is fresh


def make_cache(w, **kw):
    ws, bs = w.weights()
    quant = orc.QUANT_BF16 if w.dtype == configs.DTYPE_BF16 else orc.QUANT_NONE
    args = dict(block=w.block, search_range=w.range, search_kind=w.search, psnr_db=w.psnr_db,
                expire_n=w.expire_n, quant=quant)
    args.update(kw)
    return orc.OracleCache(w.width, w.height, w.layers, ws, bs, **args)


def test_identical_frames_reuse_the_cached_output():
    w = configs.WORKLOADS[2]()
    w.layers = nets.small_cnn(96, 80)
    w.width, w.height = 80, 96
    f = w.streams(1, 2).frame(0)[0][:96, :80]
    oc = make_cache(w)
    a = oc.infer_frame(f)
    b = oc.infer_frame(f)
    assert a["refreshed"] and not b["refreshed"]
    assert b["match"]["M"] == (0, 0) and b["match"]["matched"].all()
    for i, l in enumerate(w.layers):
        assert np.array_equal(a["maps"][i], b["maps"][i])
        if l["kind"] == orc.KIND_CONV:
            # everything but the border ring that touches padding was copied
            ring = i + 1 if i < 2 else None
            assert b["reused"][i][8:-8, 8:-8].all()
    assert np.array_equal(a["out"], b["out"])


def test_all_dirty_equals_full_inference_and_expiry():
    w = configs.WORKLOADS[2]()
    w.layers = nets.small_cnn(64, 64)
    w.width = w.height = 64
    sb = w.streams(1, 8)
    frames = [sb.frame(i)[0][:64, :64] for i in range(8)]
    cached = make_cache(w, expire_n=3)
    plain = make_cache(w, use_cache=False)
    noise = rng(1).integers(0, 256, size=(64, 64, 3), dtype=np.uint8)
    for i, f in enumerate(frames):
        if i == 4:
            f = noise                                   # unrelated frame: nothing can match
        a, b = cached.infer_frame(f), plain.infer_frame(f)
        assert b["refreshed"]
        if i % 3 == 0:
            # cache expiry: every N-th frame is a plain full inference
            assert a["refreshed"] and np.array_equal(a["out"], b["out"])
        elif i == 4:
            assert not a["refreshed"] and a["match"]["K"] == 0 and len(a["match"]["regions"]) == 0
            assert np.array_equal(a["out"], b["out"])    # all dirty == full fresh inference
        elif i == 5:
            assert not a["refreshed"] and len(a["match"]["regions"]) == 0   # its key is the noise frame
        else:
            assert not a["refreshed"]
            assert any(r is not None and r.any() for r in a["reused"])


def test_workload_1_end_to_end_reuse():
    w = configs.WORKLOADS[1]()
    sp = w.streams()
    oc = make_cache(w)
    a = oc.infer_frame(sp.frame(0)[0])
    b = oc.infer_frame(sp.frame(1)[0])
    regs = b["regions"][0]
    assert b["match"]["M"] == (-3, 2)
    mask = b["reused"][0].astype(bool)
    assert 0.3 < mask.mean() < 0.9
    for r in regs:
        if r["w"] == 0:
            continue
        assert r["sx"] - r["x"] == -3 and r["sy"] - r["y"] == 2
        d = b["out"][r["y"]:r["y"] + r["h"], r["x"]:r["x"] + r["w"]]
        s = a["out"][r["sy"]:r["sy"] + r["h"], r["sx"]:r["sx"] + r["w"]]
        assert np.array_equal(d, s)
    fresh = make_cache(w, use_cache=False).infer_frame(sp.frame(1)[0])["out"]
    assert np.array_equal(b["out"][~mask], fresh[~mask])
    # reused values are close to, but not the same as, fresh ones (sigma = 2 pixel noise)
    diff = np.abs(b["out"][mask] - fresh[mask])
    assert 0 < diff.max() < 0.2


def test_per_block_mode_reuses_two_motions_end_to_end():
    # left half static, right half moved by its own vector: the global mode can keep one of them only
    g = rng(12)
    w = configs.WORKLOADS[1]()                              # one 3x3 convolution on a 64x64 frame, block 8
    f0 = g.integers(0, 256, size=(64, 64, 3), dtype=np.uint8)
    f1 = f0.copy()
    f1[:, 32:] = np.roll(f0, (-2, 3), axis=(0, 1))[:, 32:]  # f1[y][x] = f0[y + 2][x - 3] on the right half
    own = make_cache(w, region_mode=orc.REGIONS_PER_BLOCK)
    glob = make_cache(w)
    a = own.infer_frame(f0)
    b = own.infer_frame(f1)
    glob.infer_frame(f0)
    c = glob.infer_frame(f1)
    vectors = {(int(r["sx"] - r["x"]), int(r["sy"] - r["y"])) for r in b["match"]["regions"]}
    assert vectors == {(0, 0), (-3, 2)}
    mask = b["reused"][0].astype(bool)
    # the global vector is the mean of the two motions and fits neither half of this noise image
    assert c["match"]["M"] == (-1, 1) and not c["reused"][0].any()
    assert mask.mean() > 0.5
    for r in b["regions"][0]:
        if r["w"] == 0:
            continue
        d = b["out"][r["y"]:r["y"] + r["h"], r["x"]:r["x"] + r["w"]]
        s = a["out"][r["sy"]:r["sy"] + r["h"], r["sx"]:r["sx"] + r["w"]]
        assert np.array_equal(d, s)
    fresh = make_cache(w, use_cache=False).infer_frame(f1)["out"]
    assert np.array_equal(b["out"][~mask], fresh[~mask])
    # exact copies of content: reused values equal fresh ones here (no noise was added)
    assert np.abs(b["out"] - fresh).max() < 1e-12


# ---------------------------------------------------------------------------
# reuse in pooling layers (Section 5: the cache mechanism extends to other layer types)
# ---------------------------------------------------------------------------
def pool_layer(hi, wi, c, k=2, s=2, p=0):
    return dict(kind=orc.KIND_MAXPOOL, kh=k, kw=k, sh=s, sw=s, ph=p, pw=p, cin=c, cout=c, relu=0, in0=-1, in1=-1,
                out_h=(hi + 2 * p - k) // s + 1, out_w=(wi + 2 * p - k) // s + 1)


def test_pool_reuse_copies_rectangles_and_pools_the_rest():
    g = rng(21)
    L = pool_layer(24, 20, 3)
    x = g.normal(size=(24, 20, 3))
    prev = g.normal(size=(12, 10, 3))
    regions = np.zeros(3, orc.REGION_DTYPE)
    regions[0] = (1, 2, 4, 3, 3, 0)
    regions[2] = (6, 7, 4, 5, 5, 6)
    out, reused = orc.pool_reuse(x, L, prev, regions)
    full = orc.maxpool(x, L)
    mask = np.zeros((12, 10), bool)
    for r in regions:
        mask[r["y"]:r["y"] + r["h"], r["x"]:r["x"] + r["w"]] = True
    assert np.array_equal(reused.astype(bool), mask)
    assert np.array_equal(out[~mask], full[~mask])
    assert np.array_equal(out[2:5, 1:5], prev[0:3, 3:7]) and np.array_equal(out[7:12, 6:10], prev[6:11, 5:9])
    a, b = orc.pool_reuse(x, L)                              # nothing cached: plain pooling
    assert np.array_equal(a, full) and not b.any()


def test_pool_reuse_is_exact_when_the_motion_is_a_multiple_of_the_stride():
    # content moved by (4, -4): multiples of the cumulative stride at both 2x2 pooling layers, so a cached pooled pixel
    # is the maximum over exactly the same conv outputs, and caching the pooling layers changes nothing in the result
    g = rng(22)
    w = configs.WORKLOADS[2]()
    w.layers = nets.small_cnn(96, 96)
    w.width = w.height = 96
    f0 = g.integers(0, 256, size=(96, 96, 3), dtype=np.uint8)
    f1 = np.roll(f0, (4, -4), axis=(0, 1))                   # f1[y][x] = f0[y - 4][x + 4]
    es = dict(search_kind=orc.SEARCH_ES, search_range=5)     # noise frames: a walk would stall, score every vector
    with_pool, without = make_cache(w, cache_pool=True, **es), make_cache(w, **es)
    with_pool.infer_frame(f0); without.infer_frame(f0)
    a, b = with_pool.infer_frame(f1), without.infer_frame(f1)
    assert a["match"]["M"] == (4, -4)
    pools = [i for i, l in enumerate(w.layers) if l["kind"] == orc.KIND_MAXPOOL]
    assert pools and all(a["reused"][i] is not None and a["reused"][i].mean() > 0.3 for i in pools)
    for ma, mb in zip(a["maps"], b["maps"]):
        assert np.array_equal(ma, mb)
    # an odd motion pairs a pooled pixel with a window shifted by one conv pixel: an approximation, like every
    # reuse across a stride (the paper's reuse in strided convolutions has the same property)
    f2 = np.roll(f0, (0, -3), axis=(0, 1))
    c1, c2 = make_cache(w, cache_pool=True, **es), make_cache(w, **es)
    c1.infer_frame(f0); c2.infer_frame(f0)
    p, q = c1.infer_frame(f2), c2.infer_frame(f2)
    assert p["match"]["M"] == (3, 0) and p["reused"][pools[0]].any()
    assert not np.array_equal(p["maps"][pools[0]], q["maps"][pools[0]])


# ---------------------------------------------------------------------------
# the remaining layer kinds of Table 2 as executable layers: LRN, concat, fully connected
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("r,alpha,beta,k", [(1, 1e-4, 0.75, 1.0), (2, 0.05, 0.75, 2.0), (0, 0.3, 0.5, 1.0)])
def test_lrn_equals_average_pooling_form(r, alpha, beta, k):
    g = rng(30 + r)
    x = g.normal(size=(11, 9, 5)) * 3.0
    L = dict(kind=orc.KIND_LRN, kh=2 * r + 1, kw=2 * r + 1, sh=1, sw=1, ph=r, pw=r, cin=5, cout=5, relu=0, in0=-1, in1=-1,
             out_h=11, out_w=9)
    got = orc.lrn(x, L, alpha, beta, k, orc.QUANT_NONE)
    t = torch.from_numpy(x).permute(2, 0, 1)[None]
    avg = F.avg_pool2d(t * t, 2 * r + 1, 1, r, count_include_pad=True)          # zero padding, divisor n^2 everywhere
    ref = (t / (k + alpha * avg) ** beta)[0].permute(1, 2, 0).numpy()
    assert np.abs(got - ref).max() < 1e-13


def test_lrn_closed_forms():
    L = dict(kind=orc.KIND_LRN, kh=3, kw=3, sh=1, sw=1, ph=1, pw=1, cin=1, cout=1, relu=0, in0=-1, in1=-1, out_h=5, out_w=5)
    x = np.full((5, 5, 1), 2.0)
    b = orc.lrn(x, L, 0.9, 0.5, 1.0, orc.QUANT_NONE)
    assert abs(b[2, 2, 0] - 2.0 / np.sqrt(1.0 + 0.9 * 4.0)) < 1e-15             # interior: mean of squares = 4
    assert abs(b[0, 0, 0] - 2.0 / np.sqrt(1.0 + 0.9 * 16.0 / 9.0)) < 1e-15      # corner: 4 of the 9 taps are inside
    assert abs(b[0, 2, 0] - 2.0 / np.sqrt(1.0 + 0.9 * 24.0 / 9.0)) < 1e-15      # edge: 6 of 9
    # the region rule and the arithmetic agree: an output pixel depends exactly on the (2r+1)^2 window
    y = x.copy(); y[4, 4, 0] = 7.0
    c = orc.lrn(y, L, 0.9, 0.5, 1.0, orc.QUANT_NONE)
    changed = np.argwhere(c[..., 0] != b[..., 0])
    assert set(map(tuple, changed)) == {(3, 3), (3, 4), (4, 3), (4, 4)}


def test_concat_and_fully_connected():
    g = rng(33)
    a, b = g.normal(size=(4, 5, 3)), g.normal(size=(4, 5, 2))
    c = orc.concat(a, b)
    assert c.shape == (4, 5, 5) and np.array_equal(c[..., :3], a) and np.array_equal(c[..., 3:], b)
    x = g.normal(size=(3, 4, 6))
    w = g.normal(size=(7, 3, 4, 6))
    bias = g.normal(size=7)
    L = dict(kind=orc.KIND_FC, kh=3, kw=4, sh=1, sw=1, ph=0, pw=0, cin=6, cout=7, relu=1, in0=-1, in1=-1, out_h=1, out_w=1)
    got = orc.fully_connected(x, L, w, bias, orc.QUANT_NONE)
    ref = F.linear(torch.from_numpy(x).reshape(1, -1), torch.from_numpy(w).reshape(7, -1), torch.from_numpy(bias)).clamp_min(0)
    assert got.shape == (1, 1, 7) and np.abs(got[0, 0] - ref[0].numpy()).max() < 1e-12


def test_graph_with_every_layer_kind_runs_and_reuses():
    w = configs.WORKLOADS[2]()
    w.layers = nets.inception_lrn_net(64, 64)
    w.width = w.height = 64
    sb = w.streams(1, 3)
    frames = [sb.frame(i)[0][:64, :64] for i in range(3)]
    cached, plain = make_cache(w), make_cache(w, use_cache=False)
    for i, f in enumerate(frames):
        a, b = cached.infer_frame(f), plain.infer_frame(f)
        assert a["out"].shape == (1, 1, 48)
        if i == 0:
            assert np.array_equal(a["out"], b["out"])
        else:
            assert a["reused"][0].any()                                          # first convolution reuses
            assert len(a["regions"][-1]) == 0 or not a["regions"][-1]["w"].any()  # Table 2: nothing reusable after FC
            assert np.abs(a["out"] - b["out"]).max() < 0.5


def test_lrn_reuse_copies_rectangles_and_normalises_the_rest():
    g = rng(35)
    L = dict(kind=orc.KIND_LRN, kh=3, kw=3, sh=1, sw=1, ph=1, pw=1, cin=2, cout=2, relu=0, in0=-1, in1=-1, out_h=9, out_w=8)
    x = g.normal(size=(9, 8, 2))
    prev = g.normal(size=(9, 8, 2))
    regions = np.zeros(2, orc.REGION_DTYPE)
    regions[1] = (2, 3, 4, 5, 1, 2)
    out, reused = orc.lrn_reuse(x, L, 0.1, 0.75, 1.0, orc.QUANT_NONE, prev, regions)
    full = orc.lrn(x, L, 0.1, 0.75, 1.0, orc.QUANT_NONE)
    mask = np.zeros((9, 8), bool); mask[3:8, 2:6] = True
    assert np.array_equal(reused.astype(bool), mask)
    assert np.array_equal(out[3:8, 2:6], prev[2:7, 1:5]) and np.array_equal(out[~mask], full[~mask])


# ---------------------------------------------------------------------------
# residual add and stand-alone ReLU (the multi-input and "others" rows of Table 2 as executable layers)
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("relu", [0, 1])
def test_add_equals_torch_float64(relu):
    g = rng(40 + relu)
    a, b = g.normal(size=(7, 5, 6)), g.normal(size=(7, 5, 6))
    ref = torch.from_numpy(a) + torch.from_numpy(b)
    if relu:
        ref = ref.clamp_min(0)
    got = orc.add(a, b, relu, orc.QUANT_NONE)
    assert np.array_equal(got, ref.numpy())                             # one float64 addition: no rounding freedom
    assert (got < 0).any() != bool(relu)
    # a swapped or dropped operand, or a ReLU applied before the sum, would show here
    a2, b2 = np.array([[[-3.0, 2.0]]]), np.array([[[1.0, -5.0]]])
    assert np.array_equal(orc.add(a2, b2, 0, orc.QUANT_NONE), [[[-2.0, -3.0]]])
    assert np.array_equal(orc.add(a2, b2, 1, orc.QUANT_NONE), [[[0.0, 0.0]]])
    assert np.array_equal(orc.add(-a2, -b2, 1, orc.QUANT_NONE), [[[2.0, 3.0]]])


def test_add_rounds_the_sum_to_bf16_once():
    # operands as a bf16 workload stores them (8 significant bits), close in magnitude: their sum is exact in
    # float32, so torch's double -> float -> bfloat16 conversion rounds only once, like the oracle
    g = rng(42)
    a = g.integers(-255, 256, size=4000) / 64.0
    b = g.integers(-255, 256, size=4000) / 32.0
    for relu in (0, 1):
        ref = torch.from_numpy(a + b)
        if relu:
            ref = ref.clamp_min(0)
        ref = ref.to(torch.bfloat16).to(torch.float64).numpy()
        assert np.array_equal(orc.add(a, b, relu, orc.QUANT_BF16), ref)
    # exact ties go to the even neighbour: 1 + 2^-8 -> 1; (1 + 2^-7) + 2^-8 -> 1 + 2^-6
    tie = orc.add(np.array([1.0, 1.0078125]), np.array([0.00390625, 0.00390625]), 0, orc.QUANT_BF16)
    assert np.array_equal(tie, [1.0, 1.015625])
    # the ReLU acts on the sum before rounding; a negative sum never rounds to a positive value
    assert np.array_equal(orc.add(np.array([-1.0]), np.array([0.99609375]), 1, orc.QUANT_BF16), [0.0])


def test_relu_layer_equals_torch():
    g = rng(43)
    x = g.normal(size=(5, 4, 3))
    assert np.array_equal(orc.relu(x), torch.from_numpy(x).clamp_min(0).numpy())
    assert np.array_equal(orc.relu(np.array([-0.5, 0.0, 2.5])), [0.0, 0.0, 2.5])
    q = orc.quant_array(x, orc.QUANT_BF16)
    assert np.array_equal(orc.quant_array(orc.relu(q), orc.QUANT_BF16), orc.relu(q))    # stored values stay stored values


def _residual_net(h, w):
    """conv 3x3 -> [branch: conv 3x3 + ReLU, conv 1x1] + skip -> add (+ReLU) -> stand-alone ReLU of a signed 1x1 conv."""
    nb = nets.NetBuilder(h, w)
    stem = nb.conv(-1, 4, 3, 1, 1, relu=1)
    b1 = nb.conv(stem, 4, 3, 1, 1, relu=1)
    b2 = nb.conv(b1, 4, 1, 1, 0, relu=0)
    s = nb.add(b2, stem, relu=1)
    lin = nb.conv(s, 5, 1, 1, 0, relu=0)
    nb.layers.append(dict(kind=orc.KIND_RELU, kh=1, kw=1, sh=1, sw=1, ph=0, pw=0, cin=5, cout=5, relu=0, in0=lin, in1=-1,
                          out_h=h, out_w=w, groups=1))
    return nb.layers


def _torch_conv(x, w, b, p, relu):
    y = F.conv2d(x, torch.from_numpy(w).permute(0, 3, 1, 2), torch.from_numpy(b), padding=p)
    return y.clamp_min(0) if relu else y


def test_residual_block_through_the_cache_equals_torch_float64():
    h, w_ = 24, 20
    layers = _residual_net(h, w_)
    ws, bs = nets.random_weights(layers, 7)
    oc = orc.OracleCache(w_, h, layers, ws, bs, block=8, search_range=4, search_kind=orc.SEARCH_DS)
    f = rng(44).integers(0, 256, size=(h, w_, 3), dtype=np.uint8)
    a = oc.infer_frame(f)
    x = torch.from_numpy(f.astype(np.float64) / 255.0).permute(2, 0, 1)[None]
    W = [None if v is None else np.asarray(v, np.float64) for v in ws]
    Bv = [None if v is None else np.asarray(v, np.float64) for v in bs]
    stem = _torch_conv(x, W[0], Bv[0], 1, True)
    b1 = _torch_conv(stem, W[1], Bv[1], 1, True)
    b2 = _torch_conv(b1, W[2], Bv[2], 0, False)
    s = (b2 + stem).clamp_min(0)                      # in0 = branch, in1 = skip
    lin = _torch_conv(s, W[4], Bv[4], 0, False)
    out = lin.clamp_min(0)
    for got, ref in ((a["maps"][3], s), (a["maps"][4], lin), (a["maps"][5], out)):
        assert np.abs(got - ref[0].permute(1, 2, 0).numpy()).max() < 1e-12
    assert (a["maps"][4] < 0).any() and not (a["maps"][5] < 0).any()
    # the same frame again: both inputs of the add carry the same rectangles, so its output is reusable and the
    # whole network output is the cached one
    b = oc.infer_frame(f)
    assert not b["refreshed"] and b["regions"][3]["w"].any()
    for ma, mb in zip(a["maps"], b["maps"]):
        assert np.array_equal(ma, mb)
