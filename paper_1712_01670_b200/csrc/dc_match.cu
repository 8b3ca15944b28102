// Image block matching (Section 4, Steps 1-5) on the GPU.  Integer arithmetic only.
//
//   k_search   Step 2: one warp per block; the block of the current frame sits in shared
//              memory, candidates of the previous frame are fetched as unaligned 32-bit words
//              (two aligned loads + funnel shift), |a-b| per byte by vabsdiff4, squares summed
//              by dp4a, warp-reduced.  Candidates are ordered by (SSE, |dx|+|dy|, dy, dx).
//              Blocks that pass the PSNR bound add their vector to the Step 3 sums.
//   k_verify   Steps 3-4: rounds the mean vector M, scores every block at M.
//   k_merge    Step 5: maximal horizontal runs, merged vertically when spans are identical,
//              emitted in (y, x) order by a block-wide scan.
#include "dc_common.cuh"

namespace {

constexpr int WARPS = 8;
constexpr int MAX_ROW_WORDS = 24;       // block <= 32 px -> 96 bytes per row

struct MatchArgs {
    const uint8_t* cur;  size_t cur_pitch;  size_t cur_stream;
    const uint8_t* prev; size_t prev_pitch; size_t prev_stream;
    int W, H, B, R, Gx, Gy, S, search;
    uint32_t limit[4];
    int16_t* mv; uint32_t* sse; uint8_t* matched; int32_t* acc; int32_t* gmv;
};

__device__ __forceinline__ unsigned long long cand_key(uint32_t sse, int dx, int dy)
{
    // lexicographic (SSE, |dx|+|dy|, dy, dx) packed into one integer
    return ((unsigned long long)sse << 32) | ((unsigned long long)(abs(dx) + abs(dy)) << 16) |
           ((unsigned long long)(dy + 128) << 8) | (unsigned long long)(dx + 128);
}

template <int ITERS>
struct BlockCtx {
    const uint32_t* cur_sm;     // this warp's copy of the current block, row stride MAX_ROW_WORDS
    const uint8_t* prev;        // previous frame of this stream
    size_t prev_pitch;
    int W, H, R, x0, y0, bw, bh, lane;
    int off[ITERS];             // per lane item: byte offset of (row, word) inside a candidate
    int smi[ITERS];             // index into cur_sm, -1 = no item
    uint32_t msk[ITERS];        // valid bytes of the word

    __device__ __forceinline__ void setup()
    {
        const int row_bytes = bw * 3, wpr = (row_bytes + 3) >> 2, items = bh * wpr;
#pragma unroll
        for (int it = 0; it < ITERS; ++it) {
            int item = it * 32 + lane;
            if (item < items) {
                int row = item / wpr, wi = item - row * wpr;
                int nb = row_bytes - wi * 4;
                off[it] = row * (int)prev_pitch + wi * 4;
                smi[it] = row * MAX_ROW_WORDS + wi;
                msk[it] = nb >= 4 ? 0xffffffffu : ((1u << (nb * 8)) - 1u);
            } else { off[it] = 0; smi[it] = -1; msk[it] = 0; }
        }
    }
    __device__ __forceinline__ bool valid(int dx, int dy) const
    {
        return abs(dx) <= R && abs(dy) <= R && x0 + dx >= 0 && y0 + dy >= 0 &&
               x0 + dx + bw <= W && y0 + dy + bh <= H;
    }
    // SSE of the block against the previous frame displaced by (dx, dy); same value in all lanes
    __device__ __forceinline__ uint32_t sse(int dx, int dy) const
    {
        const uint8_t* base = prev + (size_t)(y0 + dy) * prev_pitch + (size_t)(x0 + dx) * 3;
        uint32_t acc = 0;
#pragma unroll
        for (int it = 0; it < ITERS; ++it) {
            if (smi[it] >= 0) {
                const uint8_t* p = base + off[it];
                uintptr_t a = (uintptr_t)p;
                const uint32_t* q = (const uint32_t*)(a & ~(uintptr_t)3);
                uint32_t sh = ((uint32_t)a & 3u) * 8u;
                uint32_t lo = __ldg(q), hi = __ldg(q + 1);
                uint32_t pv = __funnelshift_r(lo, hi, sh) & msk[it];
                uint32_t d = __vabsdiffu4(cur_sm[smi[it]], pv);
                acc = __dp4a(d, d, acc);
            }
        }
        return __reduce_add_sync(0xffffffffu, acc);
    }
};

template <int ITERS>
__device__ __forceinline__ bool load_block(const MatchArgs& a, uint32_t* sm, BlockCtx<ITERS>& c, int& s, int& b)
{
    int warp = blockIdx.x * WARPS + (threadIdx.x >> 5);
    int per = a.Gx * a.Gy;
    if (warp >= per * a.S) return false;
    s = warp / per; b = warp - s * per;
    int by = b / a.Gx, bx = b - by * a.Gx;
    c.lane = threadIdx.x & 31;
    c.x0 = bx * a.B; c.y0 = by * a.B;
    c.bw = min(a.B, a.W - c.x0); c.bh = min(a.B, a.H - c.y0);
    c.W = a.W; c.H = a.H; c.R = a.R;
    c.prev = a.prev + (size_t)s * a.prev_stream; c.prev_pitch = a.prev_pitch;
    c.cur_sm = sm;
    c.setup();
    // the current block: byte loads (the caller's frame has no alignment or padding promise)
    const uint8_t* cur = a.cur + (size_t)s * a.cur_stream + (size_t)c.y0 * a.cur_pitch + (size_t)c.x0 * 3;
    const int row_bytes = c.bw * 3;
#pragma unroll
    for (int it = 0; it < ITERS; ++it) {
        if (c.smi[it] >= 0) {
            int row = c.smi[it] / MAX_ROW_WORDS, wi = c.smi[it] - row * MAX_ROW_WORDS;
            const uint8_t* p = cur + (size_t)row * a.cur_pitch + wi * 4;
            uint32_t v = 0;
            for (int k = 0; k < 4; ++k)
                if (wi * 4 + k < row_bytes) v |= (uint32_t)__ldg(p + k) << (8 * k);
            sm[c.smi[it]] = v;
        }
    }
    __syncwarp();
    return true;
}

__device__ __forceinline__ int limit_index(const MatchArgs& a, int bw, int bh)
{
    return (bh < a.B ? 2 : 0) + (bw < a.B ? 1 : 0);
}

template <int ITERS>
__global__ void __launch_bounds__(WARPS * 32) k_search(MatchArgs a)
{
    __shared__ uint32_t sm_all[WARPS][32 * MAX_ROW_WORDS];
    BlockCtx<ITERS> c; int s, b;
    if (!load_block<ITERS>(a, sm_all[threadIdx.x >> 5], c, s, b)) return;

    int bx_ = 0, by_ = 0;
    uint32_t bs = c.sse(0, 0);                         // the zero vector is always a candidate
    unsigned long long bk = cand_key(bs, 0, 0);
    if (a.search == DC_SEARCH_EXHAUSTIVE) {
        for (int dy = -a.R; dy <= a.R; ++dy)
            for (int dx = -a.R; dx <= a.R; ++dx) {
                if ((dx == 0 && dy == 0) || !c.valid(dx, dy)) continue;
                uint32_t v = c.sse(dx, dy);
                unsigned long long k = cand_key(v, dx, dy);
                if (k < bk) { bk = k; bs = v; bx_ = dx; by_ = dy; }
            }
    } else {
        // large diamond until its centre wins, then one small diamond
        const int lx[8] = {0, -1, 1, -2, 2, -1, 1, 0}, ly[8] = {-2, -1, -1, 0, 0, 1, 1, 2};
        const int sx[4] = {0, -1, 1, 0}, sy[4] = {-1, 0, 0, 1};
        const int max_steps = (2 * a.R + 1) * (2 * a.R + 1);   // every move strictly lowers the key
        for (int step = 0; step < max_steps; ++step) {
            int cx = bx_, cy = by_;
#pragma unroll 1
            for (int i = 0; i < 8; ++i) {
                int dx = cx + lx[i], dy = cy + ly[i];
                if (!c.valid(dx, dy)) continue;
                uint32_t v = c.sse(dx, dy);
                unsigned long long k = cand_key(v, dx, dy);
                if (k < bk) { bk = k; bs = v; bx_ = dx; by_ = dy; }
            }
            if (bx_ == cx && by_ == cy) break;
        }
        int cx = bx_, cy = by_;
#pragma unroll 1
        for (int i = 0; i < 4; ++i) {
            int dx = cx + sx[i], dy = cy + sy[i];
            if (!c.valid(dx, dy)) continue;
            uint32_t v = c.sse(dx, dy);
            unsigned long long k = cand_key(v, dx, dy);
            if (k < bk) { bk = k; bs = v; bx_ = dx; by_ = dy; }
        }
    }
    if (c.lane == 0) {
        size_t g = (size_t)s * a.Gx * a.Gy + b;
        a.mv[2 * g] = (int16_t)bx_; a.mv[2 * g + 1] = (int16_t)by_; a.sse[g] = bs;
        if (bs <= a.limit[limit_index(a, c.bw, c.bh)]) {          // PSNR > T (Step 3's set S)
            atomicAdd(&a.acc[4 * s + 0], bx_);
            atomicAdd(&a.acc[4 * s + 1], by_);
            atomicAdd(&a.acc[4 * s + 2], 1);
        }
    }
}

// mean of n values with sum `sum`, rounded to nearest, halves away from zero
__device__ __forceinline__ int round_mean(int sum, int n)
{
    int m = (2 * abs(sum) + n) / (2 * n);
    return sum < 0 ? -m : m;
}

template <int ITERS>
__global__ void __launch_bounds__(WARPS * 32) k_verify(MatchArgs a)
{
    __shared__ uint32_t sm_all[WARPS][32 * MAX_ROW_WORDS];
    BlockCtx<ITERS> c; int s, b;
    if (!load_block<ITERS>(a, sm_all[threadIdx.x >> 5], c, s, b)) return;
    int K = a.acc[4 * s + 2];
    int Mx = 0, My = 0;
    if (K > 0) { Mx = round_mean(a.acc[4 * s + 0], K); My = round_mean(a.acc[4 * s + 1], K); }
    int ok = 0;
    if (K > 0 && c.valid(Mx, My)) {
        uint32_t v = c.sse(Mx, My);
        ok = v <= a.limit[limit_index(a, c.bw, c.bh)];
    }
    if (c.lane == 0) {
        a.matched[(size_t)s * a.Gx * a.Gy + b] = (uint8_t)ok;
        if (ok) atomicAdd(&a.acc[4 * s + 3], 1);
        if (b == 0) { a.gmv[3 * s] = Mx; a.gmv[3 * s + 1] = My; a.gmv[3 * s + 2] = K; }
    }
}

// Step 5.  One CTA per stream.
__global__ void __launch_bounds__(256) k_merge(const uint8_t* matched, const int32_t* gmv, int W, int H, int B,
                                               int Gx, int Gy, int max_regions, dc_region* regions,
                                               int32_t* n_regions, int32_t* status)
{
    __shared__ int warp_sums[8];
    __shared__ int base;
    const int s = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const uint8_t* m = matched + (size_t)s * Gx * Gy;
    dc_region* out = regions + (size_t)s * max_regions;
    const int Mx = gmv[3 * s], My = gmv[3 * s + 1];
    if (tid == 0) base = 0;
    __syncthreads();
    auto same_run = [&](int r, int c0, int c1) {      // row r has a maximal run exactly [c0, c1)
        if (c0 > 0 && m[r * Gx + c0 - 1]) return false;
        if (c1 < Gx && m[r * Gx + c1]) return false;
        for (int c = c0; c < c1; ++c) if (!m[r * Gx + c]) return false;
        return true;
    };
    for (int start = 0; start < Gx * Gy; start += 256) {
        int b = start + tid, head = 0, c1 = 0, h = 0, r = 0, c0 = 0;
        if (b < Gx * Gy) {
            r = b / Gx; c0 = b - r * Gx;
            if (m[b] && (c0 == 0 || !m[b - 1])) {
                c1 = c0; while (c1 < Gx && m[r * Gx + c1]) ++c1;
                if (!(r > 0 && same_run(r - 1, c0, c1))) {
                    head = 1; h = 1;
                    while (r + h < Gy && same_run(r + h, c0, c1)) ++h;
                }
            }
        }
        // ordered compaction: exclusive scan of `head` over the 256 threads
        unsigned bal = __ballot_sync(0xffffffffu, head);
        int pre = __popc(bal & ((1u << lane) - 1u));
        if (lane == 0) warp_sums[wid] = __popc(bal);
        __syncthreads();
        int woff = 0, total = 0;
        for (int i = 0; i < 8; ++i) { if (i < wid) woff += warp_sums[i]; total += warp_sums[i]; }
        int idx = base + woff + pre;
        if (head) {
            if (idx < max_regions) {
                int x = c0 * B, y = r * B;
                int x1 = min(c1 * B, W), y1 = min((r + h) * B, H);
                dc_region g = { x, y, x1 - x, y1 - y, x + Mx, y + My };
                out[idx] = g;
            } else {
                atomicExch(status, (int)DC_ERR_OVERFLOW);
            }
        }
        __syncthreads();
        if (tid == 0) base += total;
        __syncthreads();
    }
    if (tid == 0) n_regions[s] = min(base, max_regions);
}

template <int ITERS>
int launch_all(dc_cache* c, MatchArgs& a)
{
    int warps = a.S * a.Gx * a.Gy;
    int grid = dc_div_up(warps, WARPS);
    { dc_prof_scope ps(c, DC_ST_SEARCH); k_search<ITERS><<<grid, WARPS * 32, 0, c->stream>>>(a); }
    { dc_prof_scope ps(c, DC_ST_VERIFY); k_verify<ITERS><<<grid, WARPS * 32, 0, c->stream>>>(a); }
    return 0;
}

}  // namespace

int dc_launch_match(dc_cache* c, const uint8_t* frame, size_t pitch)
{
    MatchArgs a;
    a.cur = frame; a.cur_pitch = pitch; a.cur_stream = pitch * (size_t)c->cfg.height;
    a.prev = c->key; a.prev_pitch = c->key_pitch; a.prev_stream = c->key_pitch * (size_t)c->cfg.height;
    a.W = c->cfg.width; a.H = c->cfg.height; a.B = c->cfg.block; a.R = c->cfg.range;
    a.Gx = c->Gx; a.Gy = c->Gy; a.S = c->S; a.search = c->cfg.search;
    for (int i = 0; i < 4; ++i) a.limit[i] = c->sse_limit[i];
    a.mv = c->blk_mv; a.sse = c->blk_sse; a.matched = c->matched; a.acc = c->mv_acc; a.gmv = c->gmv;
    DC_CUDA(cudaMemsetAsync(c->mv_acc, 0, sizeof(int32_t) * 4 * c->S, c->stream));
    int row_words = (a.B * 3 + 3) / 4, iters = dc_div_up(a.B * row_words, 32);
    if (iters <= 2) launch_all<2>(c, a);
    else if (iters <= 3) launch_all<3>(c, a);
    else if (iters <= 6) launch_all<6>(c, a);
    else if (iters <= 12) launch_all<12>(c, a);
    else launch_all<24>(c, a);
    {
        dc_prof_scope ps(c, DC_ST_MERGE);
        k_merge<<<c->S, 256, 0, c->stream>>>(c->matched, c->gmv, a.W, a.H, a.B, a.Gx, a.Gy, c->max_regions,
                                             c->regions0, c->n_regions, c->status);
    }
    c->launches += 3;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}
