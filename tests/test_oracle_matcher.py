"""Pins for the oracle's block matcher (Section 4, Steps 1-5).

Each test ties the oracle to something other than itself: a brute-force
numpy search, the PSNR definition evaluated in floating point, constructed
frames whose answer is known in closed form, and structural invariants.
"""
import itertools
import math

import numpy as np
import pytest

from oracle import deepcache_oracle as orc
from paper_1712_01670_b200.synth import configs, streams


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def brute_sse(cur, prev, x0, y0, bw, bh, dx, dy):
    H, W = cur.shape[:2]
    if x0 + dx < 0 or y0 + dy < 0 or x0 + dx + bw > W or y0 + dy + bh > H:
        return None
    a = cur[y0:y0 + bh, x0:x0 + bw].astype(np.int64)
    b = prev[y0 + dy:y0 + dy + bh, x0 + dx:x0 + dx + bw].astype(np.int64)
    return int(((a - b) ** 2).sum())


def brute_es(cur, prev, B, R):
    H, W = cur.shape[:2]
    Gx, Gy = -(-W // B), -(-H // B)
    mv = np.zeros((Gy, Gx, 2), np.int16)
    sse = np.zeros((Gy, Gx), np.uint32)
    for by, bx in itertools.product(range(Gy), range(Gx)):
        x0, y0 = bx * B, by * B
        bw, bh = min(B, W - x0), min(B, H - y0)
        best = None
        for dy in range(-R, R + 1):
            for dx in range(-R, R + 1):
                s = brute_sse(cur, prev, x0, y0, bw, bh, dx, dy)
                if s is None:
                    continue
                key = (s, abs(dx) + abs(dy), dy, dx)
                if best is None or key < best:
                    best = key
        mv[by, bx] = (best[3], best[2])
        sse[by, bx] = best[0]
    return mv, sse


@pytest.mark.parametrize("shape,B,R", [((20, 24), 8, 3), ((19, 23), 8, 4), ((16, 16), 5, 2), ((9, 30), 16, 6)])
def test_es_equals_brute_force(shape, B, R):
    g = rng(11)
    prev = g.integers(0, 256, size=shape + (3,), dtype=np.uint8)
    cur = np.roll(prev, (1, -2), axis=(0, 1))
    cur[3:9, 4:11] = g.integers(0, 256, size=(6, 7, 3))
    mv, sse = orc.search(cur, prev, B, R, orc.SEARCH_ES)
    mv_b, sse_b = brute_es(cur, prev, B, R)
    assert np.array_equal(mv, mv_b)
    assert np.array_equal(sse, sse_b)


def test_block_sse_equals_numpy_and_rejects_outside():
    g = rng(5)
    cur = g.integers(0, 256, size=(21, 17, 3), dtype=np.uint8)
    prev = g.integers(0, 256, size=(21, 17, 3), dtype=np.uint8)
    for (x0, y0, bw, bh, dx, dy) in [(0, 0, 8, 8, 0, 0), (8, 8, 8, 8, -3, 2), (16, 16, 1, 5, -1, 0),
                                     (0, 0, 8, 8, -1, 0), (16, 16, 1, 5, 1, 0), (8, 16, 8, 5, 0, 1)]:
        assert orc.block_sse(cur, prev, x0, y0, bw, bh, dx, dy) == brute_sse(cur, prev, x0, y0, bw, bh, dx, dy)
    # maximum possible SSE of a 16x16 block fits the uint32 the matcher reports
    a = np.zeros((16, 16, 3), np.uint8)
    b = np.full((16, 16, 3), 255, np.uint8)
    assert orc.block_sse(a, b, 0, 0, 16, 16, 0, 0) == 16 * 16 * 3 * 255 ** 2 < 2 ** 32


def test_ties_prefer_small_motion():
    # a constant frame: every candidate has SSE 0, the zero vector must win
    f = np.full((32, 32, 3), 77, np.uint8)
    for kind in (orc.SEARCH_ES, orc.SEARCH_DS):
        mv, sse = orc.search(f, f, 8, 4, kind)
        assert not mv.any() and not sse.any()
    # horizontally periodic pattern (period 4): dx = -4, 0, +4 tie at SSE 0 -> zero vector;
    # after a shift by one pixel the candidates dx = +1 and dx = -3 tie -> smaller |dx| wins
    x = np.arange(32)
    row = ((x % 4) * 60).astype(np.uint8)
    prev = np.repeat(np.repeat(row[None, :, None], 32, 0), 3, 2)
    cur = np.roll(prev, -1, axis=1)            # cur[x] = prev[x+1]  ->  dx = +1
    mv, sse = orc.search(cur, prev, 8, 4, orc.SEARCH_ES)
    inner = mv[:, 1:-1]
    assert (inner[..., 0] == 1).all() and (inner[..., 1] == 0).all() and not sse[:, 1:-1].any()


def test_identical_frames_match_everywhere():
    w = configs.WORKLOADS[2]()
    f = w.streams(1, 2).frame(0)[0]
    for kind in (orc.SEARCH_ES, orc.SEARCH_DS):
        R = 3 if kind == orc.SEARCH_ES else 16
        m = orc.match_blocks(f, f, 16, R, kind, 20.0)
        assert not m["mv"].any() and not m["sse"].any()
        assert m["M"] == (0, 0) and m["K"] == m["matched"].size
        assert m["matched"].all()
        assert len(m["regions"]) == 1
        assert tuple(m["regions"][0]) == (0, 0, 227, 227, 0, 0)     # clipped edge blocks keep the whole frame


def test_psnr_limit_closed_form_at_20db():
    # T = 20: PSNR > 20  <=>  255^2 n / SSE > 100  <=>  100 SSE < 65025 n
    for n in (1, 3, 27, 48, 75, 192, 300, 768, 16 * 3 * 3, 16 * 8 * 3):
        L = orc.psnr_limit(n, 20.0)
        assert 100 * L < 65025 * n <= 100 * (L + 1)
    # zero error has infinite PSNR and passes
    assert orc.lib().orc_psnr_pass(0, 768, 20.0) == 1


@pytest.mark.parametrize("T", [15.0, 20.0, 23.5, 30.0, 37.25])
def test_psnr_limit_against_floating_point_psnr(T):
    g = rng(3)
    for n in (27, 192, 300, 768):
        L = orc.psnr_limit(n, T)
        for sse in set(int(v) for v in g.integers(1, 4 * L + 8, size=200)) | {L, L + 1}:
            psnr = 10.0 * math.log10(65025.0 * n / sse)
            if abs(psnr - T) < 1e-9:
                continue                      # on the boundary floating point cannot decide
            assert (psnr > T) == (sse <= L), (n, sse, psnr, L)


def test_mean_mv_rounding_and_threshold():
    W = H = 32
    B = 8
    mv = np.zeros((4, 4, 2), np.int16)
    sse = np.zeros((4, 4), np.uint32)
    lim = orc.psnr_limit(192, 20.0)
    # 3 blocks pass with dx = 1,1,2 -> 4/3 -> 1 ; dy = -1,-2,-2 -> -5/3 -> -2
    sse[:] = lim + 1
    for k, (dx, dy) in enumerate([(1, -1), (1, -2), (2, -2)]):
        mv[0, k] = (dx, dy)
        sse[0, k] = lim - k
    mv[1, 1] = (9, 9)                           # fails the test: ignored
    assert orc.mean_mv(mv, sse, W, H, B, 20.0) == (1, -2, 3)
    # exact halves round away from zero: sums +-3 over 2 blocks -> +-2 (not 1.5 -> 1)
    sse[:] = lim + 1
    mv[:] = 0
    mv[0, 0] = (1, -1); mv[0, 1] = (2, -2); sse[0, 0] = sse[0, 1] = 0
    assert orc.mean_mv(mv, sse, W, H, B, 20.0) == (2, -2, 2)
    # nothing passes: K = 0, no motion, and Step 4 matches nothing
    sse[:] = lim + 1
    assert orc.mean_mv(mv, sse, W, H, B, 20.0) == (0, 0, 0)
    f = np.zeros((H, W, 3), np.uint8)
    assert not orc.verify(f, f, B, 0, 0, 0, 20.0).any()


def test_shifted_pair_recovers_global_motion():
    """Workload 1 by construction: frame1[y][x] = frame0[y+2][x-3], so every interior block's
    match in the previous frame sits at (dx, dy) = (-3, +2); the redrawn 16x16 patch is uniform
    noise against uniform noise (about 7.7 dB) and must fail Step 4, while sigma = 2 noise alone
    (about 42 dB) passes."""
    w = configs.WORKLOADS[1]()
    sp = w.streams().streams[0]
    f0, f1 = sp.frame(0), sp.frame(1)
    m = orc.match_blocks(f1, f0, 8, 8, orc.SEARCH_ES, 20.0)
    assert m["M"] == (-3, 2)
    B = 8
    for by in range(8):
        for bx in range(8):
            x0, y0 = bx * B, by * B
            inside = x0 - 3 >= 0 and y0 + 2 + B <= 64
            touches_patch = not (x0 + B <= sp.patch_x or x0 >= sp.patch_x + 16 or
                                 y0 + B <= sp.patch_y or y0 >= sp.patch_y + 16)
            if not inside:
                assert m["matched"][by, bx] == 0        # displaced block leaves the frame
            elif not touches_patch:
                assert m["matched"][by, bx] == 1
                assert tuple(m["mv"][by, bx]) == (-3, 2)
            elif (x0 >= sp.patch_x and x0 + B <= sp.patch_x + 16 and
                  y0 >= sp.patch_y and y0 + B <= sp.patch_y + 16):
                assert m["matched"][by, bx] == 0        # wholly redrawn block


def test_verify_is_sse_at_global_offset():
    g = rng(8)
    prev = g.integers(0, 256, size=(40, 48, 3), dtype=np.uint8)
    cur = np.roll(prev, (-2, 3), axis=(0, 1))       # cur[y][x] = prev[y+2][x-3]
    cur[8:16, 16:24] = 255 - cur[8:16, 16:24]
    matched = orc.verify(cur, prev, 8, -3, 2, 5, 20.0)
    for by in range(5):
        for bx in range(6):
            s = brute_sse(cur, prev, bx * 8, by * 8, 8, 8, -3, 2)
            expect = s is not None and 100 * s < 65025 * 192
            assert matched[by, bx] == int(expect)
    assert matched[1, 2] == 0 and matched[2, 3] == 1


def ds_walk_reference(cur, prev, x0, y0, bw, bh, R):
    """Independent restatement of the large/small diamond walk on a precomputed SSE surface."""
    surf = {}
    for dy in range(-R, R + 1):
        for dx in range(-R, R + 1):
            s = brute_sse(cur, prev, x0, y0, bw, bh, dx, dy)
            if s is not None:
                surf[(dx, dy)] = (s, abs(dx) + abs(dy), dy, dx)
    c = (0, 0)
    while True:
        pts = [c] + [(c[0] + a, c[1] + b) for a, b in
                     ((0, -2), (0, 2), (-2, 0), (2, 0), (-1, -1), (1, -1), (-1, 1), (1, 1))]
        best = min((p for p in pts if p in surf), key=lambda p: surf[p])
        if best == c:
            break
        c = best
    pts = [c] + [(c[0] + a, c[1] + b) for a, b in ((0, -1), (0, 1), (-1, 0), (1, 0))]
    best = min((p for p in pts if p in surf), key=lambda p: surf[p])
    return best, surf[best][0], surf


def test_diamond_search_invariants():
    w = configs.WORKLOADS[2]()
    sb = w.streams(1, 6)
    B, R = 16, 6
    for i in (1, 3, 5):
        cur, prev = sb.frame(i)[0][:80, :96], sb.frame(i - 1)[0][:80, :96]
        mv, sse = orc.search(cur, prev, B, R, orc.SEARCH_DS)
        mv_es, sse_es = orc.search(cur, prev, B, R, orc.SEARCH_ES)
        assert (np.abs(mv) <= R).all()
        assert (sse >= sse_es).all()                 # a walk can never beat the exhaustive minimum
        for by in range(5):
            for bx in range(6):
                dx, dy = (int(v) for v in mv[by, bx])
                assert orc.block_sse(cur, prev, bx * B, by * B, B, B, dx, dy) == int(sse[by, bx])
                best, s, surf = ds_walk_reference(cur, prev, bx * B, by * B, B, B, R)
                assert (dx, dy) == best and int(sse[by, bx]) == s
                # local optimality: no small-diamond neighbour of the result is better
                for a, b in ((0, -1), (0, 1), (-1, 0), (1, 0)):
                    q = (dx + a, dy + b)
                    if q in surf:
                        assert surf[(dx, dy)] < surf[q] or q == (dx, dy)


def test_diamond_equals_exhaustive_on_unimodal_surface():
    # sin(x) + sin(y) with period = block size: over a whole block the cross term cancels, so
    # SSE(dx, dy) = A(dx - sx) + B(dy - sy) with A, B increasing in |.| up to half a period.
    # On such a separable single-basin surface the diamond walk must reach the exhaustive minimum.
    y, x = np.mgrid[0:96, 0:96].astype(np.float64)
    v = 127.0 + 60.0 * np.sin(2 * np.pi * x / 16.0) + 60.0 * np.sin(2 * np.pi * y / 16.0)
    prev = np.repeat(np.rint(v).astype(np.uint8)[:, :, None], 3, 2)
    for shift in ((3, -2), (-5, 4), (0, 6), (1, 1), (-6, -6)):
        cur = np.roll(prev, (-shift[1], -shift[0]), axis=(0, 1))     # cur[y][x] = prev[y+sy][x+sx]
        ds, sse_ds = orc.search(cur, prev, 16, 6, orc.SEARCH_DS)
        es, sse_es = orc.search(cur, prev, 16, 6, orc.SEARCH_ES)
        inner = (slice(1, -1), slice(1, -1))
        assert np.array_equal(ds[inner], es[inner]) and np.array_equal(sse_ds[inner], sse_es[inner])
        assert (es[inner][..., 0] == shift[0]).all() and (es[inner][..., 1] == shift[1]).all()
        assert not sse_es[inner].any()


def cover(regions, W, H):
    m = np.zeros((H, W), np.int32)
    for r in regions:
        m[r["y"]:r["y"] + r["h"], r["x"]:r["x"] + r["w"]] += 1
    return m


def test_merge_pins():
    W, H, B = 50, 37, 10                            # ragged: last column 10 px, last row 7 px
    Gx, Gy = 5, 4
    # all matched -> one rectangle covering the frame
    r = orc.merge(np.ones((Gy, Gx), np.uint8), W, H, B, 2, -1)
    assert [tuple(v) for v in r] == [(0, 0, 50, 37, 2, -1)]
    # none matched -> nothing
    assert len(orc.merge(np.zeros((Gy, Gx), np.uint8), W, H, B, 0, 0)) == 0
    # checkerboard -> one rectangle per matched block, ordered by (y, x)
    cb = (np.add.outer(np.arange(Gy), np.arange(Gx)) % 2 == 0).astype(np.uint8)
    r = orc.merge(cb, W, H, B, 0, 0)
    assert len(r) == int(cb.sum())
    assert [(v["y"], v["x"]) for v in r] == sorted((v["y"], v["x"]) for v in r)
    assert all(v["w"] == 10 and v["h"] in (10, 7) for v in r)
    # Section 4's example: two adjacent 5x5 blocks become one 5x10 rectangle
    r = orc.merge(np.array([[1, 1]], np.uint8), 10, 5, 5, 0, 0)
    assert [tuple(v) for v in r] == [(0, 0, 10, 5, 0, 0)]
    # runs merge vertically only when their column spans are identical
    m = np.array([[1, 1, 1, 0, 1],
                  [1, 1, 1, 0, 1],
                  [1, 1, 0, 0, 1],
                  [0, 1, 1, 1, 1]], np.uint8)
    r = orc.merge(m, W, H, B, 1, 1)
    assert [tuple(v)[:4] for v in r] == [(0, 0, 30, 20), (40, 0, 10, 30), (0, 20, 20, 10), (10, 30, 40, 7)]
    assert all(v["sx"] == v["x"] + 1 and v["sy"] == v["y"] + 1 for v in r)


def test_merge_covers_exactly_the_matched_blocks():
    g = rng(21)
    for trial in range(20):
        W, H, B = int(g.integers(17, 90)), int(g.integers(17, 90)), int(g.integers(4, 17))
        Gx, Gy = -(-W // B), -(-H // B)
        m = (g.random((Gy, Gx)) < 0.6).astype(np.uint8)
        r = orc.merge(m, W, H, B, 0, 0)
        c = cover(r, W, H)
        expect = np.kron(m, np.ones((B, B), np.int32))[:H, :W]
        assert np.array_equal(c, expect)             # disjoint (no pixel counted twice) and complete


def test_k_skip_searches_every_kth_block_only():
    """Section 4: with k-skip only blocks on every k-th row and column are searched; k = 2 leaves a quarter."""
    w = configs.WORKLOADS[2]()
    sb = w.streams(1, 3)
    cur, prev = sb.frame(2)[0], sb.frame(1)[0]
    mv1, sse1 = orc.search(cur, prev, 16, 8, orc.SEARCH_DS)
    for k in (2, 3):
        mvk, ssek = orc.search(cur, prev, 16, 8, orc.SEARCH_DS, skip_k=k)
        Gy, Gx = sse1.shape
        on = np.zeros((Gy, Gx), bool)
        on[::k, ::k] = True
        assert np.array_equal(mvk[on], mv1[on]) and np.array_equal(ssek[on], sse1[on])     # searched blocks: unchanged
        assert (ssek[~on] == 2 ** 32 - 1).all() and not mvk[~on].any()                     # the rest: not searched
        if k == 2:
            assert on.sum() == -(-Gy // 2) * -(-Gx // 2)                                   # about a quarter of the blocks
        # Step 3 averages the searched blocks only
        lim = orc.psnr_limit(16 * 16 * 3, 20.0)
        full = (np.arange(Gy)[:, None] < Gy - 1) & (np.arange(Gx)[None, :] < Gx - 1)      # unclipped blocks share one bound
        sel = on & full & (sse1 <= lim)
        Mx, My, K = orc.mean_mv(mvk, ssek, 227, 227, 16, 20.0)
        edge_pass = 0
        for by in range(Gy):
            for bx in range(Gx):
                if on[by, bx] and not full[by, bx]:
                    bw, bh = min(16, 227 - bx * 16), min(16, 227 - by * 16)
                    edge_pass += int(ssek[by, bx] <= orc.psnr_limit(bw * bh * 3, 20.0))
        assert K == int(sel.sum()) + edge_pass
    # k-skip changes Step 2 and 3 only: Step 4 still scores every block at M
    m = orc.match_blocks(cur, prev, 16, 8, orc.SEARCH_DS, 20.0, skip_k=2)
    want = orc.verify(cur, prev, 16, m["M"][0], m["M"][1], m["K"], 20.0)
    assert np.array_equal(m["matched"], want)


# ---------------------------------------------------------------------------
# three step search (Section 7.5 names it as an alternative unit for Step 2)
# ---------------------------------------------------------------------------
def smooth_pair(shift, size=96):
    """prev = sin(x) + sin(y) with period 16; cur[y][x] = prev[y + sy][x + sx] (see the diamond pin above)."""
    y, x = np.mgrid[0:size, 0:size].astype(np.float64)
    v = 127.0 + 60.0 * np.sin(2 * np.pi * x / 16.0) + 60.0 * np.sin(2 * np.pi * y / 16.0)
    prev = np.repeat(np.rint(v).astype(np.uint8)[:, :, None], 3, 2)
    return np.roll(prev, (-shift[1], -shift[0]), axis=(0, 1)), prev


def test_three_step_with_range_1_is_the_exhaustive_search():
    # R = 1: the only pass has S = 1, and the centre plus its eight neighbours are the whole +-1 window
    g = rng(41)
    prev = g.integers(0, 256, size=(37, 45, 3), dtype=np.uint8)
    cur = g.integers(0, 256, size=(37, 45, 3), dtype=np.uint8)
    cur[5:30, 4:40] = prev[6:31, 3:39]                       # part of the frame moved by (-1, +1)
    for B in (8, 10, 16):
        tss, sse_tss = orc.search(cur, prev, B, 1, orc.SEARCH_TSS)
        es, sse_es = orc.search(cur, prev, B, 1, orc.SEARCH_ES)
        assert np.array_equal(tss, es) and np.array_equal(sse_tss, sse_es)


@pytest.mark.parametrize("shift", [(3, -2), (-5, 4), (0, 6), (7, 7), (-7, 1), (1, 1), (0, 0)])
def test_three_step_reaches_the_minimum_of_a_separable_basin(shift):
    # steps 4, 2, 1 reach every displacement up to 7; on the separable single-basin surface each pass
    # moves to the grid point nearest the true shift on both axes, so the result is the exhaustive one
    cur, prev = smooth_pair(shift)
    tss, sse_tss = orc.search(cur, prev, 16, 7, orc.SEARCH_TSS)
    es, sse_es = orc.search(cur, prev, 16, 7, orc.SEARCH_ES)
    inner = (slice(1, -1), slice(1, -1))
    assert (es[inner][..., 0] == shift[0]).all() and (es[inner][..., 1] == shift[1]).all()
    assert np.array_equal(tss[inner], es[inner]) and not sse_tss[inner].any()


def test_three_step_first_step_rule():
    # R = 8 still starts at S = 4 (2 * 8 - 1 > 8), so a shift of 8 is out of reach although inside the
    # window; R = 15 starts at 8 and reaches it.  The pattern's period is 32 here so that 8 is unambiguous.
    y, x = np.mgrid[0:128, 0:128].astype(np.float64)
    v = 127.0 + 60.0 * np.sin(2 * np.pi * x / 32.0) + 60.0 * np.sin(2 * np.pi * y / 32.0)
    prev = np.repeat(np.rint(v).astype(np.uint8)[:, :, None], 3, 2)
    cur = np.roll(prev, (0, -8), axis=(0, 1))                # content shift (8, 0)
    inner = (slice(1, -1), slice(1, -1))
    es, _ = orc.search(cur, prev, 32, 8, orc.SEARCH_ES)
    assert (es[inner][..., 0] == 8).all() and (es[inner][..., 1] == 0).all()
    t8, s8 = orc.search(cur, prev, 32, 8, orc.SEARCH_TSS)
    assert (t8[inner][..., 0] == 7).all() and (t8[inner][..., 1] == 0).all() and s8[inner].all()
    t15, s15 = orc.search(cur, prev, 32, 15, orc.SEARCH_TSS)
    assert (t15[inner][..., 0] == 8).all() and (t15[inner][..., 1] == 0).all() and not s15[inner].any()


def tss_walk_reference(cur, prev, x0, y0, bw, bh, R):
    """Independent restatement on a precomputed SSE surface: nine-point passes with halving step."""
    surf = {}
    for dy in range(-R, R + 1):
        for dx in range(-R, R + 1):
            s = brute_sse(cur, prev, x0, y0, bw, bh, dx, dy)
            if s is not None:
                surf[(dx, dy)] = (s, abs(dx) + abs(dy), dy, dx)
    step = max(p for p in (1, 2, 4, 8, 16, 32, 64) if 2 * p - 1 <= R)
    c, visited = (0, 0), {(0, 0)}
    while step >= 1:
        pts = [(c[0] + i * step, c[1] + j * step) for j in (-1, 0, 1) for i in (-1, 0, 1)]
        visited.update(p for p in pts if p in surf)
        c = min((p for p in pts if p in surf), key=lambda p: surf[p])
        step //= 2
    return c, surf[c][0], visited


def test_three_step_invariants_on_video_frames():
    w = configs.WORKLOADS[2]()
    sb = w.streams(1, 6)
    B = 16
    for R, first in ((6, 2), (16, 8)):
        for i in (1, 4):
            cur, prev = sb.frame(i)[0][:80, :96], sb.frame(i - 1)[0][:80, :96]
            mv, sse = orc.search(cur, prev, B, R, orc.SEARCH_TSS)
            _, sse_es = orc.search(cur, prev, B, R, orc.SEARCH_ES)
            assert (np.abs(mv) <= 2 * first - 1).all()           # reach of the step sequence
            assert (sse >= sse_es).all()
            for by in range(5):
                for bx in range(6):
                    dx, dy = (int(v) for v in mv[by, bx])
                    assert orc.block_sse(cur, prev, bx * B, by * B, B, B, dx, dy) == int(sse[by, bx])
                    best, s, visited = tss_walk_reference(cur, prev, bx * B, by * B, B, B, R)
                    assert (dx, dy) == best and int(sse[by, bx]) == s
                    assert len(visited) <= 1 + 8 * (first.bit_length())     # 9 points, then 8 new ones per pass


# ---------------------------------------------------------------------------
# per-block region mode: every rectangle carries the vector of its own blocks
# ---------------------------------------------------------------------------
def merge_own_reference(matched, mv, W, H, B):
    """Independent restatement: label runs per row, then chain runs with equal (columns, vector) downwards."""
    Gy, Gx = matched.shape
    runs = []                                               # per row: list of (c0, c1, dx, dy)
    for r in range(Gy):
        row, c = [], 0
        while c < Gx:
            if not matched[r, c]:
                c += 1
                continue
            c0, v = c, tuple(mv[r, c])
            while c < Gx and matched[r, c] and tuple(mv[r, c]) == v:
                c += 1
            row.append((c0, c, v[0], v[1]))
        runs.append(row)
    out = []
    for r in range(Gy):
        for run in runs[r]:
            if r > 0 and run in runs[r - 1]:
                continue                                    # continues the rectangle above
            h = 1
            while r + h < Gy and run in runs[r + h]:
                h += 1
            x, y = run[0] * B, r * B
            x1, y1 = min(run[1] * B, W), min((r + h) * B, H)
            out.append((x, y, x1 - x, y1 - y, x + run[2], y + run[3]))
    return sorted(out, key=lambda t: (t[1], t[0]))


def test_merge_own_equals_global_merge_when_all_vectors_agree():
    g = rng(8)
    W, H, B = 75, 52, 10
    Gx, Gy = 8, 6
    matched = (g.random((Gy, Gx)) < 0.7).astype(np.uint8)
    mv = np.zeros((Gy, Gx, 2), np.int16)
    mv[..., 0], mv[..., 1] = 3, -2
    a = orc.merge_own(matched, mv, W, H, B)
    b = orc.merge(matched, W, H, B, 3, -2)
    assert [tuple(v) for v in a] == [tuple(v) for v in b]


def test_merge_own_pins():
    W, H, B = 40, 30, 10
    mv = np.zeros((3, 4, 2), np.int16)
    mv[:, :2] = (2, 0)                                      # left half moves by (2, 0), right half by (-3, 1)
    mv[:, 2:] = (-3, 1)
    r = orc.merge_own(np.ones((3, 4), np.uint8), mv, W, H, B)
    assert [tuple(v) for v in r] == [(0, 0, 20, 30, 2, 0), (20, 0, 20, 30, 17, 1)]
    # same columns, vector changes between rows 1 and 2: the rectangle is cut there
    mv2 = np.zeros((3, 4, 2), np.int16)
    mv2[2] = (1, 1)
    r = orc.merge_own(np.ones((3, 4), np.uint8), mv2, W, H, B)
    assert [tuple(v) for v in r] == [(0, 0, 40, 20, 0, 0), (0, 20, 40, 10, 1, 21)]
    # a single odd block splits its row into three runs and breaks the column chains through it
    mv3 = np.zeros((3, 4, 2), np.int16)
    mv3[1, 1] = (0, -1)
    r = orc.merge_own(np.ones((3, 4), np.uint8), mv3, W, H, B)
    assert [tuple(v) for v in r] == [(0, 0, 40, 10, 0, 0), (0, 10, 10, 10, 0, 10), (10, 10, 10, 10, 10, 9),
                                     (20, 10, 20, 10, 20, 10), (0, 20, 40, 10, 0, 20)]


def test_merge_own_equals_reference_and_covers_matched_blocks():
    g = rng(9)
    for trial in range(40):
        Gx, Gy, B = int(g.integers(1, 9)), int(g.integers(1, 8)), int(g.integers(4, 17))
        W, H = Gx * B - int(g.integers(0, B)), Gy * B - int(g.integers(0, B))
        matched = (g.random((Gy, Gx)) < 0.75).astype(np.uint8)
        mv = g.integers(-1, 1, size=(Gy, Gx, 2)).astype(np.int16)      # few distinct vectors: long runs and chains
        r = orc.merge_own(matched, mv, W, H, B)
        assert [tuple(v) for v in r] == merge_own_reference(matched, mv, W, H, B)
        m = cover(r, W, H)
        expect = np.kron(matched, np.ones((B, B), np.int32))[:H, :W]
        assert np.array_equal(m, expect)                                # disjoint, exactly the matched blocks
        for v in r:                                                     # every block inside carries the rectangle's vector
            blk = mv[v["y"] // B:-(-(v["y"] + v["h"]) // B), v["x"] // B:-(-(v["x"] + v["w"]) // B)]
            assert (blk[..., 0] == v["sx"] - v["x"]).all() and (blk[..., 1] == v["sy"] - v["y"]).all()


def test_accept_own_is_the_step_2_psnr_test():
    g = rng(10)
    prev = g.integers(0, 256, size=(48, 64, 3), dtype=np.uint8)
    cur = prev.copy()
    cur[:, 32:] = np.roll(prev, (-1, 3), axis=(0, 1))[:, 32:]           # right half: cur[y][x] = prev[y + 1][x - 3]
    cur[16:32, 0:16] = g.integers(0, 256, size=(16, 16, 3))             # one block replaced by noise
    m = orc.match_blocks(cur, prev, 16, 4, orc.SEARCH_ES, 20.0, region_mode=orc.REGIONS_PER_BLOCK)
    lim = 16 * 16 * 3 * 65025 // 100                                    # 20 dB: SSE < n * 650.25
    assert np.array_equal(m["matched"], (m["sse"] <= lim).astype(np.uint8))
    assert m["matched"][1, 0] == 0 and m["matched"].sum() == 9          # bottom right row would leave the frame
    regs = [tuple(v) for v in m["regions"]]
    assert (0, 0, 32, 16, 0, 0) in regs                                 # left half above the noise block, unmoved
    assert (32, 0, 32, 32, 29, 1) in regs                               # right half with its own vector
    # the global mode keeps one vector only: with two motions it loses one half
    g0 = orc.match_blocks(cur, prev, 16, 4, orc.SEARCH_ES, 20.0)
    assert g0["matched"].sum() < m["matched"].sum()
    # k-skip: blocks that were not searched have no vector of their own and stay unmatched
    k = orc.match_blocks(cur, prev, 16, 4, orc.SEARCH_ES, 20.0, skip_k=2, region_mode=orc.REGIONS_PER_BLOCK)
    assert not k["matched"][1::2].any() and not k["matched"][:, 1::2].any() and k["matched"][0, 0]
