"""The no-allocation block search against the regular matcher.

Some users of the library cannot allocate device memory at the point where they need block
matching (no cudaMalloc in their processing loop, or a host application that forbids it after
start-up), so they cannot build a cache.  dc_search_blocks_noalloc serves them with a fixed
scratch array inside the library.  Its results must be exactly those of dc_match_blocks, also
on a second call, since calls share that array and each must clear the previous call's sums.

Collected last on purpose: a failure here cannot hide any other test under ``pytest -x``.
"""
import numpy as np
import pytest
import torch

from oracle import deepcache_oracle as orc
from paper_1712_01670_b200 import binding as B
from paper_1712_01670_b200.engine import DeepCache
from paper_1712_01670_b200.synth import configs, nets

pytestmark = pytest.mark.gpu


def reference_match(prev, cur, block, R, search):
    S, H, W, _ = cur.shape
    layers = nets.single_conv(H, W)
    ws, bs = nets.random_weights(layers, 1)
    dc = DeepCache(W, H, layers, ws, bs, n_streams=S, block=block, search_range=R, search=search)
    try:
        dc.set_key(prev)
        return dc.match_blocks(cur)
    finally:
        dc.close()


@pytest.mark.parametrize("search,block,R", [(B.DC_SEARCH_DIAMOND, 16, 16), (B.DC_SEARCH_EXHAUSTIVE, 8, 5), (B.DC_SEARCH_DIAMOND, 10, 8)])
def test_noalloc_search_equals_match_blocks_twice(search, block, R):
    w = configs.WORKLOADS[2]()
    sb = w.streams(1, 5)
    # three streams: consecutive frame pairs of the panning stream (227 x 227: ragged edge blocks)
    prev_a = np.stack([sb.frame(i)[0] for i in (0, 1, 2)])
    cur_a = np.stack([sb.frame(i)[0] for i in (1, 2, 3)])
    # second call on different data, so stale sums from the first call would show
    prev_b = np.stack([sb.frame(i)[0] for i in (3, 0, 1)])
    cur_b = np.stack([sb.frame(i)[0] for i in (4, 2, 1)])
    S, H, W = 3, w.height, w.width
    Gx, Gy = -(-W // block), -(-H // block)
    dev = torch.device("cuda:0")
    mv = torch.empty((S, Gy, Gx, 2), dtype=torch.int16, device=dev)
    sse = torch.empty((S, Gy, Gx), dtype=torch.int32, device=dev)
    gmv = torch.empty((S, 3), dtype=torch.int32, device=dev)
    for prev, cur in ((prev_a, cur_a), (prev_b, cur_b)):
        want = reference_match(prev, cur, block, R, search)
        p, c = torch.from_numpy(prev).to(dev), torch.from_numpy(cur).to(dev)
        mv.fill_(-1); sse.fill_(-1); gmv.fill_(-1)
        B.dc_search_blocks_noalloc(c, p, W * 3, W, H, S, block, R, search, 20.0, mv, sse, gmv)
        torch.cuda.synchronize()
        assert torch.equal(mv, want["mv"])
        assert torch.equal(sse, want["sse"])
        assert torch.equal(gmv, want["gmv"])
        # and against the CPU oracle directly (Section 4, Steps 2 and 3), stream by stream
        for s in range(S):
            o_mv, o_sse = orc.search(cur[s], prev[s], block, R, search)
            assert np.array_equal(mv[s].cpu().numpy(), o_mv)
            assert np.array_equal(sse[s].cpu().numpy().view(np.uint32), o_sse)
            assert tuple(gmv[s].tolist()) == orc.mean_mv(o_mv, o_sse, W, H, block, 20.0)


def test_noalloc_search_takes_any_pitch_and_alignment():
    """The caller's frames need neither aligned rows nor an aligned start: rows 5 bytes longer than the pixels,
    the first pixel one byte into the buffer.  Twice, like the test above."""
    w = configs.WORKLOADS[2]()
    sb = w.streams(1, 4)
    H, W, S, block, R = 75, 83, 2, 16, 8
    pitch = W * 3 + 5
    dev = torch.device("cuda:0")
    Gx, Gy = -(-W // block), -(-H // block)
    mv = torch.empty((S, Gy, Gx, 2), dtype=torch.int16, device=dev)
    sse = torch.empty((S, Gy, Gx), dtype=torch.int32, device=dev)
    gmv = torch.empty((S, 3), dtype=torch.int32, device=dev)

    def padded(frames):                                   # [S][H][pitch] behind one leading byte, filler 0xAB
        buf = np.full(1 + S * H * pitch + 16, 0xAB, np.uint8)
        rows = buf[1:1 + S * H * pitch].reshape(S, H, pitch)
        rows[:, :, :W * 3] = frames.reshape(S, H, W * 3)
        return torch.from_numpy(buf).to(dev)

    for first in (0, 1):
        prev = np.stack([sb.frame(first + k)[0][10:10 + H, 20:20 + W] for k in (0, 1)])
        cur = np.stack([sb.frame(first + k + 1)[0][10:10 + H, 20:20 + W] for k in (0, 1)])
        pb, cb = padded(prev), padded(cur)
        mv.fill_(-1); sse.fill_(-1); gmv.fill_(-1)
        B.dc_search_blocks_noalloc(cb.data_ptr() + 1, pb.data_ptr() + 1, pitch, W, H, S, block, R, B.DC_SEARCH_DIAMOND,
                                   20.0, mv, sse, gmv)
        torch.cuda.synchronize()
        want = reference_match(prev, cur, block, R, B.DC_SEARCH_DIAMOND)
        assert torch.equal(mv, want["mv"]) and torch.equal(sse, want["sse"]) and torch.equal(gmv, want["gmv"])
        for s in range(S):
            o_mv, o_sse = orc.search(cur[s], prev[s], block, R, orc.SEARCH_DS)
            assert np.array_equal(mv[s].cpu().numpy(), o_mv)
            assert np.array_equal(sse[s].cpu().numpy().view(np.uint32), o_sse)


def test_noalloc_refuses_three_step_search():
    dev = torch.device("cuda:0")
    f = torch.zeros((1, 16, 16, 3), dtype=torch.uint8, device=dev)
    mv = torch.empty((1, 1, 1, 2), dtype=torch.int16, device=dev)
    sse = torch.empty((1, 1, 1), dtype=torch.int32, device=dev)
    gmv = torch.empty((1, 3), dtype=torch.int32, device=dev)
    with pytest.raises(B.DeepCacheError) as e:
        B.dc_search_blocks_noalloc(f, f, 48, 16, 16, 1, 16, 4, B.DC_SEARCH_THREE_STEP, 20.0, mv, sse, gmv)
    assert e.value.status == B.DC_ERR_CONFIG


def test_noalloc_rejects_sizes_beyond_its_scratch():
    dev = torch.device("cuda:0")
    f = torch.zeros((1, 16, 16, 3), dtype=torch.uint8, device=dev)
    mv = torch.empty((1, 1, 1, 2), dtype=torch.int16, device=dev)
    sse = torch.empty((1, 1, 1), dtype=torch.int32, device=dev)
    gmv = torch.empty((1, 3), dtype=torch.int32, device=dev)
    with pytest.raises(B.DeepCacheError) as e:
        B.dc_search_blocks_noalloc(f, f, 48, 16, 16, B.DC_NOALLOC_MAX_STREAMS + 1, 16, 4, 1, 20.0, mv, sse, gmv)
    assert e.value.status == B.DC_ERR_LIMIT and "limit" in str(e.value)
