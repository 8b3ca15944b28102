"""Pins for the oracle's region propagation (Section 5, Table 2, Fig. 7)."""
import os

import numpy as np
import pytest

from oracle import deepcache_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "erosion_examples.txt")


def layer(kind, k=1, s=1, p=0, out_h=0, out_w=0, in0=-1, in1=-1):
    return dict(kind=kind, kh=k, kw=k, sh=s, sw=s, ph=p, pw=p, cin=1, cout=1, relu=0,
                in0=in0, in1=in1, out_h=out_h, out_w=out_w)


def regs(*rows):
    a = np.zeros(len(rows), orc.REGION_DTYPE)
    for i, r in enumerate(rows):
        a[i] = tuple(r)
    return a


def golden_rows():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, ksp, rin, rout = (v.strip() for v in line.split("|"))
            rows.append((name, tuple(map(int, ksp.split())), tuple(map(int, rin.split())),
                         tuple(map(int, rout.split()))))
    return rows


@pytest.mark.parametrize("name,ksp,rin,rout", golden_rows())
def test_printed_examples(name, ksp, rin, rout):
    k, s, p = ksp
    L = layer(orc.KIND_CONV, k, s, p, 1000, 1000)
    out = orc.propagate_layer(L, 1000, 1000, regs(rin + rin[:2]))[0]
    assert (out["x"], out["y"], out["w"], out["h"]) == rout
    # a pooling layer with the same parameters erodes the same way (one Table 2 row for both)
    L = layer(orc.KIND_MAXPOOL, k, s, p, 1000, 1000)
    out = orc.propagate_layer(L, 1000, 1000, regs(rin + rin[:2]))[0]
    assert (out["x"], out["y"], out["w"], out["h"]) == rout


def test_fig7_mapping_and_relu():
    # current (100,100,100,40) -> cached (120,120,100,40) through conv k11 s2 p5, then ReLU
    r = regs((100, 100, 100, 40, 120, 120))
    out = orc.propagate_layer(layer(orc.KIND_CONV, 11, 2, 5, 150, 150), 300, 300, r)
    assert tuple(out[0]) == (53, 53, 45, 15, 63, 63)
    out2 = orc.propagate_layer(layer(orc.KIND_RELU), 150, 150, out)
    assert tuple(out2[0]) == tuple(out[0])
    # the pooling layer that follows in the figure (k3 s2 p1) shrinks it again
    out3 = orc.propagate_layer(layer(orc.KIND_MAXPOOL, 3, 2, 1, 75, 75), 150, 150, out2)
    assert 0 < out3[0]["w"] < out[0]["w"] and 0 < out3[0]["h"] < out[0]["h"]


def test_table2_other_rows():
    r = regs((10, 12, 30, 20, 13, 11), (0, 0, 4, 4, 0, 0))
    # LRN radius r: (x + r, y + r, w - 2r, h - 2r); equals a k = 2r+1, s = 1, p = r window layer
    lrn = orc.propagate_layer(layer(orc.KIND_LRN, 5, 1, 2, 64, 64), 64, 64, r)
    assert tuple(lrn[0]) == (12, 14, 26, 16, 15, 13)
    assert tuple(lrn[1]) == (0, 0, 0, 0, 0, 0)              # 4 - 2*2 = 0: vanished
    conv = orc.propagate_layer(layer(orc.KIND_CONV, 5, 1, 2, 64, 64), 64, 64, r)
    assert tuple(conv[0]) == tuple(lrn[0])
    # fully connected / softmax: (0, 0, 0, 0)
    fc = orc.propagate_layer(layer(orc.KIND_FC), 64, 64, r)
    assert all(tuple(v) == (0, 0, 0, 0, 0, 0) for v in fc)
    # concat / add: the overlapped region; displacement must agree
    a = regs((10, 10, 20, 20, 12, 9), (0, 0, 8, 8, 1, 1), (5, 5, 5, 5, 5, 5))
    b = regs((15, 5, 20, 20, 17, 4), (0, 0, 8, 8, 2, 1), (20, 20, 5, 5, 20, 20))
    for kind in (orc.KIND_CONCAT, orc.KIND_ADD):
        o = orc.propagate_layer(layer(kind), 64, 64, a, b)
        assert tuple(o[0]) == (15, 10, 15, 15, 17, 9)
        assert tuple(o[1]) == (0, 0, 0, 0, 0, 0)             # displacements differ
        assert tuple(o[2]) == (0, 0, 0, 0, 0, 0)             # no overlap


def reusable_by_tracing(in_mask, k, s, p, n_out):
    """Boolean dependency tracing on one axis pair: an output is reusable iff every input tap of
    its window is inside the map and marked reusable (padding counts as not reusable)."""
    H, W = in_mask.shape
    out = np.zeros((n_out[0], n_out[1]), bool)
    for oy in range(n_out[0]):
        for ox in range(n_out[1]):
            ok = True
            for ky in range(k):
                for kx in range(k):
                    iy, ix = oy * s - p + ky, ox * s - p + kx
                    if iy < 0 or iy >= H or ix < 0 or ix >= W or not in_mask[iy, ix]:
                        ok = False
            out[oy, ox] = ok
    return out


def mask_of(regions, H, W):
    m = np.zeros((H, W), bool)
    for r in regions:
        m[r["y"]:r["y"] + r["h"], r["x"]:r["x"] + r["w"]] = True
    return m


def test_erosion_equals_dependency_tracing_through_a_stack():
    g = np.random.Generator(np.random.PCG64(4))
    stack = [(3, 1, 1), (2, 2, 0), (5, 1, 2), (3, 2, 1), (11, 4, 0), (1, 2, 0)]
    for trial in range(30):
        H, W = int(g.integers(30, 70)), int(g.integers(30, 70))
        x, y = int(g.integers(0, W - 8)), int(g.integers(0, H - 8))
        w, h = int(g.integers(1, W - x + 1)), int(g.integers(1, H - y + 1))
        r = regs((x, y, w, h, x, y))
        m = mask_of(r, H, W)
        hh, ww = H, W
        for (k, s, p) in [stack[i] for i in g.permutation(len(stack))[:3]]:
            oh, ow = (hh + 2 * p - k) // s + 1, (ww + 2 * p - k) // s + 1
            if oh <= 0 or ow <= 0:
                break
            r = orc.propagate_layer(layer(orc.KIND_CONV, k, s, p, oh, ow), hh, ww, r)
            m = reusable_by_tracing(m, k, s, p, (oh, ow))
            assert np.array_equal(mask_of(r, oh, ow), m), (trial, k, s, p)
            hh, ww = oh, ow


def test_multi_layer_erosion_equals_receptive_field_closed_form():
    # composed stack: stride S = prod s_i, field R = 1 + sum (k_i - 1) prod_{j<i} s_j,
    # padding P = sum p_i prod_{j<i} s_j.  Output o is reusable iff [oS - P, oS - P + R - 1]
    # lies inside [x, x + w - 1].
    stack = [(3, 1, 1), (3, 1, 1), (2, 2, 0), (3, 1, 1), (3, 2, 1), (5, 1, 2)]
    S, R, P = 1, 1, 0
    for (k, s, p) in stack:
        R += (k - 1) * S
        P += p * S
        S *= s
    n = 400
    for (x, w) in [(0, 400), (37, 111), (100, 33), (5, 390), (64, 64), (17, R), (17, R - 1)]:
        r = regs((x, x, w, w, x, x))
        size = n
        for (k, s, p) in stack:
            out = (size + 2 * p - k) // s + 1
            r = orc.propagate_layer(layer(orc.KIND_CONV, k, s, p, out, out), size, size, r)
            size = out
        expect = [o for o in range(size) if o * S - P >= x and o * S - P + R - 1 <= x + w - 1]
        if not expect:
            assert r[0]["w"] == 0 and r[0]["h"] == 0
        else:
            assert (r[0]["x"], r[0]["w"]) == (expect[0], len(expect))
            assert (r[0]["y"], r[0]["h"]) == (expect[0], len(expect))


def test_never_below_printed_width_formula():
    # Table 2 prints w' = floor((w - k)/s); the interval form used here is never smaller and
    # at most one larger, and agrees with the printed x' = ceil((x + p)/s)
    g = np.random.Generator(np.random.PCG64(9))
    for _ in range(500):
        k, s = int(g.integers(1, 12)), int(g.integers(1, 5))
        p = int(g.integers(0, k))
        x, w = int(g.integers(0, 200)), int(g.integers(k, 200))
        o = orc.propagate_layer(layer(orc.KIND_CONV, k, s, p, 500, 500), 500, 500, regs((x, x, w, w, x, x)))[0]
        printed = (w - k) // s
        if o["w"] > 0:
            assert o["x"] == -(-(x + p) // s)
            assert printed <= o["w"] <= printed + 1
        else:
            assert printed <= 0


def test_cached_side_uses_same_transform_and_smaller_size():
    # motion not divisible by the stride: the two sides can differ by one; the smaller size is kept
    L = layer(orc.KIND_CONV, 3, 2, 1, 100, 100)
    for (x, sx, w) in [(10, 13, 40), (11, 14, 41), (10, 11, 7), (0, 3, 200 - 3)]:
        o = orc.propagate_layer(L, 200, 200, regs((x, x, w, w, sx, sx)))[0]
        d = orc.propagate_layer(L, 200, 200, regs((x, x, w, w, x, x)))[0]
        c = orc.propagate_layer(L, 200, 200, regs((sx, sx, w, w, sx, sx)))[0]
        assert (o["x"], o["sx"]) == (d["x"], c["x"])
        assert o["w"] == min(d["w"], c["w"]) and o["h"] == min(d["h"], c["h"])
        assert o["sx"] + o["w"] <= 100 and o["x"] + o["w"] <= 100


def test_resize_rule_equals_span_tracing():
    g = np.random.Generator(np.random.PCG64(2))
    for (n_in, n_out) in [(1920, 224), (1080, 224), (100, 30), (64, 64), (17, 5)]:
        for _ in range(40):
            x = int(g.integers(0, n_in - 1))
            w = int(g.integers(1, n_in - x + 1))
            L = layer(orc.KIND_RESIZE_AREA, out_h=n_out, out_w=n_out)
            o = orc.propagate_layer(L, n_in, n_in, regs((x, x, w, w, x, x)))[0]
            expect = []
            for q in range(n_out):
                lo, hi = (q * n_in) // n_out, -(-((q + 1) * n_in) // n_out) - 1
                if lo >= x and hi <= x + w - 1:
                    expect.append(q)
            if expect:
                assert (o["x"], o["w"]) == (expect[0], len(expect))
            else:
                assert o["w"] == 0


def test_propagate_walks_the_graph():
    from paper_1712_01670_b200.synth import nets
    layers = nets.resnet50_trunk(224, 224)
    whole = regs((0, 0, 224, 224, 0, 0))
    per = orc.propagate(layers, (224, 224), whole)
    # zero motion over the whole frame: only the border erodes (padding is not reusable), the
    # displacement stays zero, and deep 7x7 maps may lose everything (cache erosion, Section 2)
    for l, r in zip(layers, per):
        assert r[0]["sx"] == r[0]["x"] and r[0]["sy"] == r[0]["y"]
        assert 0 <= r[0]["x"] and r[0]["x"] + r[0]["w"] <= l["out_w"]
    assert all(r[0]["w"] > 0 for r in per[:30])
    stem = per[0][0]
    assert (stem["x"], stem["w"]) == (2, 109)        # 7x7 s2 p3 on 224: outputs 2..110 see no padding
    # odd motion: the first residual add (stride 1 everywhere) keeps the region ...
    moved = regs((16, 16, 160, 160, 19, 17))
    per = orc.propagate(layers, (224, 224), moved)
    adds = [i for i, l in enumerate(layers) if l["kind"] == nets.KIND_ADD]
    assert per[adds[0]][0]["w"] > 0
    # ... and a region is dropped at an add whose two inputs disagree on the displacement
    a, b = layers[adds[3]]["in0"], layers[adds[3]]["in1"]
    ra, rb = per[a][0], per[b][0]
    if ra["w"] > 0 and rb["w"] > 0 and (ra["sx"] - ra["x"], ra["sy"] - ra["y"]) != (rb["sx"] - rb["x"], rb["sy"] - rb["y"]):
        assert per[adds[3]][0]["w"] == 0
