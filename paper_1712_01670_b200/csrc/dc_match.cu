// Image block matching (Section 4, Steps 1-5) on the GPU.  Integer arithmetic only.
//
//   k_search   Step 2: one warp per block; the block of the current frame sits in shared
//              memory, candidates of the previous frame are fetched as unaligned 32-bit words
//              (two aligned loads + funnel shift), |a-b| per byte by vabsdiff4, squares summed
//              by dp4a, warp-reduced.  Candidates are ordered by (SSE, |dx|+|dy|, dy, dx).
//              Blocks that pass the PSNR bound add their vector to the Step 3 sums.
//   k_search_dsw  Step 2 for 16-pixel blocks with diamond search (the common case): one CTA per 8 x 2
//              blocks, the previous frame's window staged once in shared memory as one word per pixel; one
//              warp per block, lane 2r + h scoring every other pixel of block row r, so that loads are free of
//              bank conflicts and of byte realignment; points already scored by the previous diamond are
//              skipped (they cannot win).  Walks that leave the window continue in k_search_dsw_long with
//              private windows.
//   k_search_tss16q  Step 2 for 16-pixel blocks with three step search: the same lane layout, one window that
//              covers the whole reach of the search.
//   k_verify   Steps 3-4: rounds the mean vector M, scores every block at M (reusing the Step 2
//              score when the block's own best vector is M); k_verify16_prep / k_verify16_list for 16-pixel blocks.
//   k_merge_runs, k_merge   Step 5: maximal horizontal runs per block row, merged vertically when the
//              spans are identical, emitted in (y, x) order by a CTA-wide ordered compaction.
#include "dc_common.cuh"

namespace {

constexpr int WARPS = 8;
constexpr int MAX_ROW_WORDS = 24;       // block <= 32 px -> 96 bytes per row

struct MatchArgs {
    const uint8_t* cur;  size_t cur_pitch;  size_t cur_stream;
    const uint8_t* prev; size_t prev_pitch; size_t prev_stream;
    int W, H, B, R, Gx, Gy, S, search, skip_k, region_mode;
    int edge_only;                       // generic search: 1 = only blocks clipped by the frame edge, 2 = only blocks clipped in width (the rest has a fast kernel)
    uint32_t limit[4];
    int16_t* mv; uint32_t* sse; uint8_t* matched; int32_t* acc; int32_t* gmv;
    int32_t* status;                     // device status word: a walk ended by its step limit records DC_ERR_TIMEOUT
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
    if ((a.edge_only == 1 && c.bw == a.B && c.bh == a.B) || (a.edge_only == 2 && c.bw == a.B)) return false;
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
    if (a.skip_k > 1 && ((b % a.Gx) % a.skip_k != 0 || (b / a.Gx) % a.skip_k != 0)) {
        // Section 4, k-skip: this block is not searched and takes no part in Step 3
        if (c.lane == 0) {
            size_t g = (size_t)s * a.Gx * a.Gy + b;
            a.mv[2 * g] = 0; a.mv[2 * g + 1] = 0; a.sse[g] = 0xffffffffu;
        }
        return;
    }

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
    } else if (a.search == DC_SEARCH_THREE_STEP) {
        // nine-point passes with step S0, S0/2, ..., 1; S0 = largest power of two with 2 S0 - 1 <= R
        int step = a.R < 1 ? 0 : 1;
        while (4 * step - 1 <= a.R) step *= 2;
        for (; step >= 1; step >>= 1) {
            const int cx = bx_, cy = by_;
#pragma unroll 1
            for (int i = 0; i < 9; ++i) {
                if (i == 4) continue;
                const int dx = cx + (i % 3 - 1) * step, dy = cy + (i / 3 - 1) * step;
                if (!c.valid(dx, dy)) continue;
                uint32_t v = c.sse(dx, dy);
                unsigned long long k = cand_key(v, dx, dy);
                if (k < bk) { bk = k; bs = v; bx_ = dx; by_ = dy; }
            }
        }
    } else {
        // large diamond until its centre wins, then one small diamond
        const int lx[8] = {0, -1, 1, -2, 2, -1, 1, 0}, ly[8] = {-2, -1, -1, 0, 0, 1, 1, 2};
        const int sx[4] = {0, -1, 1, 0}, sy[4] = {-1, 0, 0, 1};
        const int max_steps = (2 * a.R + 1) * (2 * a.R + 1);   // every move strictly lowers the key: never reached
        bool settled = false;
        for (int step = 0; step < max_steps && !settled; ++step) {
            int cx = bx_, cy = by_;
#pragma unroll 1
            for (int i = 0; i < 8; ++i) {
                int dx = cx + lx[i], dy = cy + ly[i];
                if (!c.valid(dx, dy)) continue;
                uint32_t v = c.sse(dx, dy);
                unsigned long long k = cand_key(v, dx, dy);
                if (k < bk) { bk = k; bs = v; bx_ = dx; by_ = dy; }
            }
            settled = bx_ == cx && by_ == cy;
        }
        if (!settled && c.lane == 0) atomicExch(a.status, (int)DC_ERR_TIMEOUT);   // the limit ended the walk: result not valid
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

// Per-block mode, in place of Step 4: a searched block is accepted with its own vector when that match passed
// the PSNR test of Step 2.  One thread per block.  The global vector is still reported.
__global__ void k_accept_own(MatchArgs a)
{
    const int per = a.Gx * a.Gy;
    const int gi = blockIdx.x * blockDim.x + threadIdx.x;
    if (gi >= per * a.S) return;
    const int s = gi / per, b = gi - s * per, by = b / a.Gx, bx = b - by * a.Gx;
    const int bw = min(a.B, a.W - bx * a.B), bh = min(a.B, a.H - by * a.B);
    const uint32_t v = a.sse[gi];
    const int ok = v != 0xffffffffu && v <= a.limit[limit_index(a, bw, bh)];
    a.matched[gi] = (uint8_t)ok;
    if (ok) atomicAdd(&a.acc[4 * s + 3], 1);
    if (b == 0) {
        const int K = a.acc[4 * s + 2];
        a.gmv[3 * s] = K > 0 ? round_mean(a.acc[4 * s + 0], K) : 0;
        a.gmv[3 * s + 1] = K > 0 ? round_mean(a.acc[4 * s + 1], K) : 0;
        a.gmv[3 * s + 2] = K;
    }
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
        const size_t g = (size_t)s * a.Gx * a.Gy + b;
        // Section 4's second acceleration: a score that Step 2 already computed for the pair (block, block + M)
        // is taken over instead of being recomputed -- exact when the block's best vector is M itself
        uint32_t v = (a.mv[2 * g] == Mx && a.mv[2 * g + 1] == My && a.sse[g] != 0xffffffffu) ? a.sse[g] : c.sse(Mx, My);
        ok = v <= a.limit[limit_index(a, c.bw, c.bh)];
    }
    if (c.lane == 0) {
        a.matched[(size_t)s * a.Gx * a.Gy + b] = (uint8_t)ok;
        if (ok) atomicAdd(&a.acc[4 * s + 3], 1);
        if (b == 0) { a.gmv[3 * s] = Mx; a.gmv[3 * s + 1] = My; a.gmv[3 * s + 2] = K; }
    }
}

// Step 5, part 1: for every block that starts a maximal horizontal run of matched blocks, the column
// where the run ends; 0 for every other block (an end is never 0).  One thread per block; the forward
// scan of a run start stays inside one row of bytes (cache hits after the first touch).
__global__ void k_merge_runs(const uint8_t* matched, const int16_t* mv, int Gx, int total, uint16_t* run_end)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= total) return;
    const int c = b % Gx;
    uint16_t e = 0;
    if (mv == nullptr) {
        if (matched[b] && (c == 0 || !matched[b - 1])) {
            int j = c + 1;
            while (j < Gx && matched[b - c + j]) ++j;
            e = (uint16_t)j;
        }
    } else if (matched[b]) {
        // per-block mode: a run also ends where the vector changes
        const uint32_t* v = (const uint32_t*)mv;                  // (dx, dy) as one word
        const uint32_t mine = v[b];
        if (c == 0 || !matched[b - 1] || v[b - 1] != mine) {
            int j = c + 1;
            while (j < Gx && matched[b - c + j] && v[b - c + j] == mine) ++j;
            e = (uint16_t)j;
        }
    }
    run_end[b] = e;
}

// Step 5, part 2: a run continues the rectangle above it only when the run directly above starts and
// ends at the same columns; every other run heads a rectangle that extends down while that holds.
// One CTA per stream; heads are emitted in (y, x) order by a CTA-wide ordered compaction.
// In per-block mode (mv != nullptr) the run above, and the runs below, must also carry the same vector,
// and the rectangle's source is displaced by that vector instead of the global one.
__global__ void __launch_bounds__(1024) k_merge(const uint16_t* run_end, const int16_t* mv, const int32_t* gmv, int W, int H, int B,
                                                int Gx, int Gy, int max_regions, dc_region* regions,
                                                int32_t* n_regions, int32_t* status)
{
    __shared__ int warp_sums[32];
    __shared__ int base;
    const int s = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const uint16_t* e = run_end + (size_t)s * Gx * Gy;
    const uint32_t* v = mv ? (const uint32_t*)mv + (size_t)s * Gx * Gy : nullptr;
    dc_region* out = regions + (size_t)s * max_regions;
    int Mx = gmv[3 * s], My = gmv[3 * s + 1];
    if (tid == 0) base = 0;
    __syncthreads();
    for (int start = 0; start < Gx * Gy; start += 1024) {
        const int b = start + tid;
        int head = 0, c1 = 0, h = 0, r = 0, c0 = 0;
        if (b < Gx * Gy) {
            r = b / Gx; c0 = b - r * Gx;
            c1 = e[b];
            if (c1 != 0 && !(r > 0 && e[b - Gx] == c1 && (!v || v[b - Gx] == v[b]))) {
                head = 1; h = 1;
                while (r + h < Gy && e[b + h * Gx] == c1 && (!v || v[b + h * Gx] == v[b])) ++h;
            }
        }
        // ordered compaction: exclusive scan of `head` over the 1024 threads
        const unsigned bal = __ballot_sync(0xffffffffu, head);
        const int pre = __popc(bal & ((1u << lane) - 1u));
        if (lane == 0) warp_sums[wid] = __popc(bal);
        __syncthreads();
        int woff = 0, total = 0;
        for (int i = 0; i < 32; ++i) { const int v = warp_sums[i]; if (i < wid) woff += v; total += v; }
        const int idx = base + woff + pre;
        if (head) {
            if (idx < max_regions) {
                const int x = c0 * B, y = r * B;
                const int x1 = min(c1 * B, W), y1 = min((r + h) * B, H);
                if (mv) { Mx = mv[2 * ((size_t)s * Gx * Gy + b)]; My = mv[2 * ((size_t)s * Gx * Gy + b) + 1]; }
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

// ---------------------------------------------------------------------------------------------
// Fast Steps 2 and 4: 16-pixel blocks, diamond search
// ---------------------------------------------------------------------------------------------

// NR rows (48 bytes each) of the current block per lane, masked for clipped edge blocks.
template <int NR>
struct RowCtx {
    uint32_t cw[NR][12];
    int row_bytes;                                                 // bw * 3: bytes of a block row (48 unless clipped)
    // mask of the valid bytes of word j of a clipped row
    __device__ __forceinline__ uint32_t word_mask(int j) const
    {
        const int nb = row_bytes - 4 * j;
        return nb >= 4 ? 0xffffffffu : (nb <= 0 ? 0u : ((1u << (8 * nb)) - 1u));
    }
    bool clipped, row_on[NR];
    // cur_rows[k]: address of row k of this lane (16-byte aligned in the library's frame copy)
    __device__ __forceinline__ void load(const uint8_t* const* cur_rows, int bw, const bool* on)
    {
        clipped = bw < 16;
        row_bytes = bw * 3;
#pragma unroll
        for (int k = 0; k < NR; ++k) {
            row_on[k] = on[k];
            const uint4* p = (const uint4*)cur_rows[k];
            uint4 v0 = make_uint4(0, 0, 0, 0), v1 = v0, v2 = v0;
            if (on[k]) { v0 = __ldg(p); v1 = __ldg(p + 1); v2 = __ldg(p + 2); }
            cw[k][0] = v0.x; cw[k][1] = v0.y; cw[k][2] = v0.z; cw[k][3] = v0.w; cw[k][4] = v1.x; cw[k][5] = v1.y;
            cw[k][6] = v1.z; cw[k][7] = v1.w; cw[k][8] = v2.x; cw[k][9] = v2.y; cw[k][10] = v2.z; cw[k][11] = v2.w;
            if (clipped) {
#pragma unroll
                for (int j = 0; j < 12; ++j) cw[k][j] &= word_mask(j);
            }
        }
    }
    // rows r, r + step, ... of the block whose top-left byte is `base`
    __device__ __forceinline__ void load_block(const uint8_t* base, size_t pitch, int r, int step, int bw, int bh)
    {
        const uint8_t* rows[NR]; bool on[NR];
#pragma unroll
        for (int k = 0; k < NR; ++k) { rows[k] = base + (size_t)(r + k * step) * pitch; on[k] = r + k * step < bh; }
        load(rows, bw, on);
    }
    // partial SSE of row k against 13 consecutive words at q, the row starting sh bits into q[0]
    template <bool CLIP = true, typename P>
    __device__ __forceinline__ uint32_t sse(int k, P q, uint32_t sh) const
    {
        uint32_t w[13];
#pragma unroll
        for (int j = 0; j < 13; ++j) w[j] = q[j];
        return sse_words<CLIP>(k, w, sh);
    }
    // the same on 13 words already in registers
    template <bool CLIP = true>
    __device__ __forceinline__ uint32_t sse_words(int k, const uint32_t (&w)[13], uint32_t sh) const
    {
        uint32_t acc[3] = {0, 0, 0};                            // three chains hide the dp4a latency
        if (!CLIP || !clipped) {
#pragma unroll
            for (int j = 0; j < 12; ++j) {
                uint32_t d = __vabsdiffu4(cw[k][j], __funnelshift_r(w[j], w[j + 1], sh));
                acc[j % 3] = __dp4a(d, d, acc[j % 3]);
            }
        } else {
#pragma unroll
            for (int j = 0; j < 12; ++j) {
                uint32_t d = __vabsdiffu4(cw[k][j], __funnelshift_r(w[j], w[j + 1], sh) & word_mask(j));
                acc[j % 3] = __dp4a(d, d, acc[j % 3]);
            }
        }
        return acc[0] + acc[1] + acc[2];
    }
};

__device__ __forceinline__ void publish_block(const MatchArgs& a, int s, size_t g, int bw, int bh, unsigned long long bk)
{
    const int fx = (int)(bk & 0xff) - 128, fy = (int)((bk >> 8) & 0xff) - 128;
    const uint32_t fs = (uint32_t)(bk >> 32);
    a.mv[2 * g] = (int16_t)fx; a.mv[2 * g + 1] = (int16_t)fy; a.sse[g] = fs;
    if (fs <= a.limit[limit_index(a, bw, bh)]) {              // PSNR > T: member of Step 3's set S
        atomicAdd(&a.acc[4 * s + 0], fx);
        atomicAdd(&a.acc[4 * s + 1], fy);
        atomicAdd(&a.acc[4 * s + 2], 1);
    }
}

// ---------------------------------------------------------------------------------------------
// Step 2 for 16-pixel blocks, diamond search: one warp per block
// ---------------------------------------------------------------------------------------------
// The previous frame's window is staged in shared memory with one 32-bit word per pixel (R, G, B, 0), so a candidate
// displaced by (dx, dy) starts at a word whatever dx is: no byte realignment, and a candidate's address is the lane's
// base plus dy * pitch + dx.  Lane 2 r + h scores pixels h, h + 2, ..., h + 14 of block row r: its 8 pixels of the
// current block stay in registers, a candidate costs 8 loads at fixed offsets, 8 absolute differences, 8 multiply-
// accumulates and one warp sum.  With a row pitch of p words, p = 2 (mod 4), the 32 lanes of a load fall in 32
// different banks for every displacement (bank = r p + h + const, and r p / 2 runs through all residues mod 16),
// so shared memory is read without conflicts, and all lanes of a warp follow the same walk, so no lane waits for
// another block.  The points of the two diamonds sit at compile-time offsets from the centre's address.
//
// Points: 0-7 the large diamond, 8 its centre, 9-12 the small diamond.
__host__ __device__ constexpr int point_x(int i)
{
    constexpr int t[13] = {0, -1, 1, -2, 2, -1, 1, 0, 0, 0, -1, 1, 0};
    return t[i];
}
__host__ __device__ constexpr int point_y(int i)
{
    constexpr int t[13] = {-2, -1, -1, 0, 0, 1, 1, 2, 0, -1, 0, 0, 1};
    return t[i];
}
constexpr int kNP[25] = {0, 0, 31, 0, 0, 0, 11, 0, 21, 0, 171, 0, 0, 0, 213, 0, 168, 0, 208, 0, 0, 0, 248, 0, 0};
// new-point masks of the 8 possible moves; a move's table index (my + 2) * 5 + (mx + 2) is always even
constexpr unsigned long long pack_moves(int first)
{
    unsigned long long r = 0;
    for (int h = first; h < first + 8 && 2 * h < 25; ++h) r |= (unsigned long long)kNP[2 * h] << (8 * (h - first));
    return r;
}
constexpr unsigned long long kMovesLo = pack_moves(0), kMovesHi = pack_moves(8);

// st: 0 walking, 1 finished, 2 the walk left the staged window (resume elsewhere), 3 no block
struct WalkState { int cx, cy, phase, st; uint32_t mask, bs, bt; };

__device__ __forceinline__ void walk_begin(WalkState& w, bool on)
{
    w.cx = 0; w.cy = 0; w.phase = 0; w.st = on ? 0 : 3;
    w.mask = on ? 0x1ffu : 0u;                                    // the centre (0, 0) and its large diamond
    w.bs = 0xffffffffu; w.bt = 0xffffffffu;
}
// points of the large diamond around a new centre that the diamond around the old one did not contain:
// the others lost to the new centre already and cannot win (mx, my: the move, one of the 8 diamond offsets)
__device__ __forceinline__ uint32_t new_points(int mx, int my)
{
    const int h = ((my + 2) * 5 + (mx + 2)) >> 1;
    return (uint32_t)((h < 8 ? kMovesLo >> (8 * h) : kMovesHi >> (8 * (h - 8))) & 0xffu);
}

// The same points for look-ups with a run-time index (the same in all lanes of a warp: one constant-cache access).
__constant__ int c_point_x[13] = {0, -1, 1, -2, 2, -1, 1, 0, 0, 0, -1, 1, 0};
__constant__ int c_point_y[13] = {-2, -1, -1, 0, 0, 1, 1, 2, 0, -1, 0, 0, 1};
// Per point and window pitch: byte offset of the point's candidate from the centre's, << 16, | the low 16 bits of the
// point's tie-key offset (py << 8) + px taken modulo 2^16.
__host__ __device__ constexpr int point_word(int i, int pitch)
{
    return (int)(((unsigned)((point_y(i) * pitch + point_x(i)) * 4) << 16) | ((unsigned)(point_y(i) * 256 + point_x(i)) & 0xffffu));
}
#define DC_POINT_ROW(p) {point_word(0, p), point_word(1, p), point_word(2, p), point_word(3, p), point_word(4, p), point_word(5, p), \
                         point_word(6, p), point_word(7, p), point_word(8, p), point_word(9, p), point_word(10, p), point_word(11, p), point_word(12, p)}

// displacements that keep the block inside the previous frame and the search range
struct WalkBounds { int dx_lo, dx_hi, dy_lo, dy_hi; };

__device__ __forceinline__ WalkBounds walk_bounds(const MatchArgs& a, int x0, int y0, int bw, int bh)
{
    WalkBounds b = {max(-a.R, -x0), min(a.R, a.W - bw - x0), max(-a.R, -y0), min(a.R, a.H - bh - y0)};
    return b;
}
// which of the 13 points around (cx, cy) are valid candidates
__device__ __forceinline__ uint32_t valid_points(int cx, int cy, const WalkBounds& b)
{
    if (cx - 2 >= b.dx_lo && cx + 2 <= b.dx_hi && cy - 2 >= b.dy_lo && cy + 2 <= b.dy_hi) return 0x1fffu;
    // near the frame's edge or the range limit (rare): a real loop, so that it is not merged into the path above
    uint32_t m = 0;
#pragma unroll 1
    for (int i = 0; i < 13; ++i) {
        const int dx = cx + c_point_x[i], dy = cy + c_point_y[i];
        if (dx >= b.dx_lo && dx <= b.dx_hi && dy >= b.dy_lo && dy <= b.dy_hi) m |= 1u << i;
    }
    return m;
}
__device__ __forceinline__ uint32_t tie_key(int dx, int dy)
{
    return ((uint32_t)(abs(dx) + abs(dy)) << 16) | ((uint32_t)(dy + 128) << 8) | (uint32_t)(dx + 128);
}

// The 8 pixels of row r (48 bytes at `row`, 16-byte aligned) that lane parity h scores, one word each.
__device__ __forceinline__ void load_lane_pixels(const uint8_t* row, int h, bool on, uint32_t (&cw)[8])
{
    uint32_t w[12];
    const uint4* p = (const uint4*)row;
    uint4 v0 = make_uint4(0, 0, 0, 0), v1 = v0, v2 = v0;
    if (on) { v0 = __ldg(p); v1 = __ldg(p + 1); v2 = __ldg(p + 2); }
    w[0] = v0.x; w[1] = v0.y; w[2] = v0.z; w[3] = v0.w; w[4] = v1.x; w[5] = v1.y; w[6] = v1.z; w[7] = v1.w;
    w[8] = v2.x; w[9] = v2.y; w[10] = v2.z; w[11] = v2.w;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        uint32_t px[2];
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const int k = 2 * j + q, wi = (3 * k) >> 2, sh = ((3 * k) & 3) * 8;      // pixel k: bytes 3k .. 3k + 2
            px[q] = (sh == 0 ? w[wi] : sh == 8 ? w[wi] >> 8 : __funnelshift_r(w[wi], w[wi + 1 < 12 ? wi + 1 : wi], sh)) & 0x00ffffffu;
        }
        cw[j] = h ? px[1] : px[0];
    }
}

// Expands 4 packed pixels (12 bytes in a, b, c) to 4 words and stores them at dst (8-byte aligned).
__device__ __forceinline__ void store_pixels4(uint32_t* dst, uint32_t a, uint32_t b, uint32_t c)
{
    const uint32_t m = 0x00ffffffu;
    *(uint2*)dst = make_uint2(a & m, __funnelshift_r(a, b, 24) & m);
    *(uint2*)(dst + 2) = make_uint2(__funnelshift_r(b, c, 16) & m, c >> 8);
}
// 4 pixels starting at pixel px0 (a multiple of 4) of frame row gy, zeros outside the frame copy
__device__ __forceinline__ void load_pixels4(const uint8_t* prev, size_t pitch, int H, int gy, int px0, uint32_t& a, uint32_t& b, uint32_t& c)
{
    a = b = c = 0;
    if (gy >= 0 && gy < H && px0 >= 0 && (size_t)px0 * 3 + 12 <= pitch) {
        const uint32_t* q = (const uint32_t*)(prev + (size_t)gy * pitch + (size_t)px0 * 3);     // px0 * 3 is a multiple of 12
        a = __ldg(q); b = __ldg(q + 1); c = __ldg(q + 2);
    }
}

// SSE of this lane's 8 pixels against the candidate whose first word for this lane is at shared-memory address p,
// summed over the warp.  Explicit shared-space loads at fixed offsets from one address register.
template <int OFF>
__device__ __forceinline__ uint32_t lds_at(uint32_t p)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1+%2];" : "=r"(v) : "r"(p), "n"(OFF) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t score_at(uint32_t p, const uint32_t (&cw)[8], bool row_on)
{
    const uint32_t w0 = lds_at<0>(p), w1 = lds_at<8>(p), w2 = lds_at<16>(p), w3 = lds_at<24>(p);
    const uint32_t w4 = lds_at<32>(p), w5 = lds_at<40>(p), w6 = lds_at<48>(p), w7 = lds_at<56>(p);
    uint32_t a0 = 0, a1 = 0, d;
    d = __vabsdiffu4(cw[0], w0); a0 = __dp4a(d, d, a0);
    d = __vabsdiffu4(cw[1], w1); a1 = __dp4a(d, d, a1);
    d = __vabsdiffu4(cw[2], w2); a0 = __dp4a(d, d, a0);
    d = __vabsdiffu4(cw[3], w3); a1 = __dp4a(d, d, a1);
    d = __vabsdiffu4(cw[4], w4); a0 = __dp4a(d, d, a0);
    d = __vabsdiffu4(cw[5], w5); a1 = __dp4a(d, d, a1);
    d = __vabsdiffu4(cw[6], w6); a0 = __dp4a(d, d, a0);
    d = __vabsdiffu4(cw[7], w7); a1 = __dp4a(d, d, a1);
    const uint32_t mine = row_on ? a0 + a1 : 0u;
    uint32_t sum;
    asm volatile("redux.sync.add.u32 %0, %1, 0xffffffff;" : "=r"(sum) : "r"(mine));
    return sum;
}

// The same with the candidate's offset from p known at compile time: the eight loads need no address arithmetic.
template <int OFF>
__device__ __forceinline__ uint32_t score_at_fixed(uint32_t p, const uint32_t (&cw)[8], bool row_on)
{
    const uint32_t w0 = lds_at<OFF>(p), w1 = lds_at<OFF + 8>(p), w2 = lds_at<OFF + 16>(p), w3 = lds_at<OFF + 24>(p);
    const uint32_t w4 = lds_at<OFF + 32>(p), w5 = lds_at<OFF + 40>(p), w6 = lds_at<OFF + 48>(p), w7 = lds_at<OFF + 56>(p);
    uint32_t a0 = 0, a1 = 0, d;
    d = __vabsdiffu4(cw[0], w0); a0 = __dp4a(d, d, a0);
    d = __vabsdiffu4(cw[1], w1); a1 = __dp4a(d, d, a1);
    d = __vabsdiffu4(cw[2], w2); a0 = __dp4a(d, d, a0);
    d = __vabsdiffu4(cw[3], w3); a1 = __dp4a(d, d, a1);
    d = __vabsdiffu4(cw[4], w4); a0 = __dp4a(d, d, a0);
    d = __vabsdiffu4(cw[5], w5); a1 = __dp4a(d, d, a1);
    d = __vabsdiffu4(cw[6], w6); a0 = __dp4a(d, d, a0);
    d = __vabsdiffu4(cw[7], w7); a1 = __dp4a(d, d, a1);
    const uint32_t mine = row_on ? a0 + a1 : 0u;
    uint32_t sum;
    asm volatile("redux.sync.add.u32 %0, %1, 0xffffffff;" : "=r"(sum) : "r"(mine));
    return sum;
}

// Scores the points of the compile-time set MASK around the centre whose candidate starts at pc: straight-line code,
// every load at a fixed offset.  Tracks the smallest SSE (ms), the point that gave it (mi) and whether two of
// the scores that mattered were equal (tie): the caller settles the rare ties with the exact order.
template <uint32_t MASK, int PITCH, int I = 0>
__device__ __forceinline__ void score_fixed_set(uint32_t pc, const uint32_t (&cw)[8], bool row_on, uint32_t& ms, int& mi, bool& tie)
{
    if constexpr (I < 13) {
        if constexpr (((MASK >> I) & 1u) != 0) {
            const uint32_t s = score_at_fixed<(point_y(I) * PITCH + point_x(I)) * 4>(pc, cw, row_on);
            tie |= s == ms;                                   // selects, no branches: the code stays straight
            mi = s < ms ? I : mi;
            ms = min(ms, s);
        }
        score_fixed_set<MASK, PITCH, I + 1>(pc, cw, row_on, ms, mi, tie);
    }
}

// One block's walk, by one warp, for as long as it stays inside the staged window.
//
// A round scores one of ten point sets around the current centre: kind 0-7, the points of the large diamond that are
// new after the move along diamond point `kind` (the others lost to the new centre already and cannot win); kind 8,
// the first round (centre and all eight points); kind 9, the small diamond.  Outside the first round the centre is
// the best point so far and bs its SSE.  When all 13 points around the centre are valid candidates the round runs
// as straight-line code for its set and decides by SSE alone: a point that beats the centre becomes the next centre
// and names the next round's kind.  Should two SSEs that matter be equal, or the frame edge or the range limit cut
// the set, the round is (re)done point by point under the full order (SSE, |dx| + |dy|, dy, dx): same result.
constexpr int KIND_FIRST = 8, KIND_SMALL = 9;
__constant__ uint32_t c_kind_mask[10] = {31u, 11u, 21u, 171u, 213u, 168u, 208u, 248u, 0x1ffu, 0x1e00u};
// diamond point of a move (mx, my), indexed by ((my + 2) * 5 + (mx + 2)) >> 1
__constant__ int c_kind_of_move[13] = {0, 0, 0, 1, 2, 3, 0, 4, 5, 6, 0, 7, 0};

struct WalkW {
    int cx, cy, kind;           // centre, and how it was reached
    uint32_t bs;                // SSE of the best point so far (the centre, after the first round)
    int nx, ny; uint32_t ns;    // on return 2: the centre the walk has chosen and not yet moved to, and its SSE
};

//   lane_base  shared-memory address of this lane's first word of the candidate at displacement (0, 0);
//              (dx, dy) is at lane_base + (dy * PITCH + dx) * 4
//   reach(x, y)  true when every point around centre (x, y) is staged
// Returns 1 when the walk has finished (result: w.cx, w.cy, w.bs), 2 when the next centre is out of reach.
template <int PITCH, typename Reach>
__device__ __forceinline__ int warp_walk(const MatchArgs& a, uint32_t lane_base, const uint32_t (&cw)[8], bool row_on,
                                         const WalkBounds& wb, WalkW& w, const Reach& reach)
{
    static __constant__ int c_points[13] = DC_POINT_ROW(PITCH);
    const int max_moves = (2 * a.R + 1) * (2 * a.R + 1);          // every move strictly lowers the key: never reached
    // all 13 points valid  <=>  cx in [dx_lo + 2, dx_hi - 2] and cy likewise: one unsigned compare per axis
    const int ix_lo = wb.dx_lo + 2, iy_lo = wb.dy_lo + 2;
    const unsigned ix_span = (unsigned)max(wb.dx_hi - 2 - ix_lo, -1), iy_span = (unsigned)max(wb.dy_hi - 2 - iy_lo, -1);
    uint32_t pc = lane_base + (uint32_t)((w.cy * PITCH + w.cx) * 4);
#pragma unroll 1
    for (int move = 0;; ++move) {
        const bool interior = wb.dx_hi - 2 >= ix_lo && wb.dy_hi - 2 >= iy_lo &&
                              (unsigned)(w.cx - ix_lo) <= ix_span && (unsigned)(w.cy - iy_lo) <= iy_span;
        uint32_t ms = 0xffffffffu; int mi = 8; bool tie = !interior;
        if (interior) {
            switch (w.kind) {
            case 0: score_fixed_set<31u, PITCH>(pc, cw, row_on, ms, mi, tie); break;
            case 1: score_fixed_set<11u, PITCH>(pc, cw, row_on, ms, mi, tie); break;
            case 2: score_fixed_set<21u, PITCH>(pc, cw, row_on, ms, mi, tie); break;
            case 3: score_fixed_set<171u, PITCH>(pc, cw, row_on, ms, mi, tie); break;
            case 4: score_fixed_set<213u, PITCH>(pc, cw, row_on, ms, mi, tie); break;
            case 5: score_fixed_set<168u, PITCH>(pc, cw, row_on, ms, mi, tie); break;
            case 6: score_fixed_set<208u, PITCH>(pc, cw, row_on, ms, mi, tie); break;
            case 7: score_fixed_set<248u, PITCH>(pc, cw, row_on, ms, mi, tie); break;
            case KIND_FIRST: score_fixed_set<0x1ffu, PITCH>(pc, cw, row_on, ms, mi, tie); break;
            default: score_fixed_set<0x1e00u, PITCH>(pc, cw, row_on, ms, mi, tie); break;
            }
            tie |= ms == w.bs;
        }
        int nx = w.cx, ny = w.cy;                                 // the best point after this round
        uint32_t ns = w.bs;
        if (!tie) {
            if (ms < w.bs) { ns = ms; nx = w.cx + c_point_x[mi]; ny = w.cy + c_point_y[mi]; }
        } else {
            // the exact order, point by point
            uint32_t m = c_kind_mask[w.kind] & valid_points(w.cx, w.cy, wb);
            uint32_t bt = w.kind == KIND_FIRST ? 0xffffffffu : tie_key(w.cx, w.cy);
            const uint32_t kc = ((uint32_t)(w.cy + 128) << 8) | (uint32_t)(w.cx + 128);  // low half of the centre's tie key
#pragma unroll 1
            while (m) {                                           // one candidate per turn; m is the same in all lanes
                const int i = __ffs(m) - 1;
                m &= m - 1;
                const int pw = c_points[i];
                const uint32_t s = score_at(pc + (uint32_t)(pw >> 16), cw, row_on);
                if (s <= ns) {
                    const uint32_t lo = (kc + (uint32_t)pw) & 0xffffu;               // ((dy + 128) << 8) | (dx + 128)
                    const int dx = (int)(lo & 0xff) - 128, dy = (int)(lo >> 8) - 128;
                    const uint32_t kt = ((uint32_t)(abs(dx) + abs(dy)) << 16) | lo;
                    if (s < ns || kt < bt) { ns = s; bt = kt; nx = dx; ny = dy; }
                }
            }
        }
        if (w.kind == KIND_SMALL) { w.cx = nx; w.cy = ny; w.bs = ns; return 1; }       // the small diamond's best is the result
        if (nx == w.cx && ny == w.cy) { w.bs = ns; w.kind = KIND_SMALL; continue; }    // centre won: small diamond, then done
        if (move >= max_moves) {                                  // a walk cut here is not valid: say so
            if ((threadIdx.x & 31) == 0) atomicExch(a.status, (int)DC_ERR_TIMEOUT);
            w.bs = ns;
            return 1;
        }
        if (!reach(nx, ny)) { w.nx = nx; w.ny = ny; w.ns = ns; return 2; }
        const int mx = nx - w.cx, my = ny - w.cy;
        w.kind = c_kind_of_move[((my + 2) * 5 + (mx + 2)) >> 1];
        pc += (uint32_t)((my * PITCH + mx) * 4);
        w.cx = nx; w.cy = ny; w.bs = ns;
    }
}

// Phase 1: one CTA per 8 x W_VS blocks, one warp per block.  The window reaches W_WRY rows above and below the tile
// and 12 pixels to its left and right (its left edge stays a multiple of 4 pixels, so that 4 pixels are 12 aligned
// bytes of the packed frame).  A walk whose next centre is out of reach is handed to phase 2.  Blocks clipped in
// width are left to the generic kernel.  Launched without k-skip only (every block is searched).
constexpr int W_VS = 2, W_WRY = 10, W_SIDE = 12;
constexpr int W_COLS = 128 + 2 * W_SIDE;                    // staged pixels per window row
constexpr int W_PITCH = 154;                                // words per window row
constexpr int W_ROWS = 16 * W_VS + 2 * W_WRY;
static_assert(W_PITCH % 4 == 2 && W_PITCH >= W_COLS && W_COLS % 4 == 0, "conflict-free pitch, whole groups of 4 pixels");

struct TileReach {
    __device__ __forceinline__ bool operator()(int cx, int cy) const { return abs(cx) + 2 <= W_SIDE && abs(cy) + 2 <= W_WRY; }
};

__global__ void __launch_bounds__(W_VS * 8 * 32, 3) k_search_dsw(MatchArgs a, uint4* long_list, int32_t* long_count)
{
    constexpr int THREADS = W_VS * 8 * 32, GROUPS = W_COLS / 4;
    constexpr int ROWS_PER_PASS = THREADS / GROUPS, PASSES = (W_ROWS + ROWS_PER_PASS - 1) / ROWS_PER_PASS;
    __shared__ __align__(16) uint32_t win[W_ROWS * W_PITCH];
    __shared__ int32_t sums[3];
    const int strip = blockIdx.x, vg = blockIdx.y, s = blockIdx.z;        // grid: strips of 8 blocks x groups of W_VS block rows x streams
    const int xs = strip * 128, yb = vg * 16 * W_VS;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, r = lane >> 1, h = lane & 1;
    const int by = vg * W_VS + (warp >> 3), bx = strip * 8 + (warp & 7);
    const int x0 = bx * 16, y0 = by * 16;
    const bool searched = bx < a.Gx && by < a.Gy && a.W - x0 >= 16;
    const int bh = searched ? min(16, a.H - y0) : 0;
    const bool row_on = r < bh;
    uint32_t cw[8];                                            // issued first: in flight while the window is staged
    load_lane_pixels(a.cur + (size_t)s * a.cur_stream + (size_t)(row_on ? y0 + r : 0) * a.cur_pitch + (size_t)(row_on ? x0 : 0) * 3,
                     h, row_on, cw);
    if (threadIdx.x < 3) sums[threadIdx.x] = 0;
    {   // the window: a thread keeps its group of 4 pixels (one column position) and goes down the rows, 13 rows apart
        const int gq = threadIdx.x % GROUPS, row0 = threadIdx.x / GROUPS, px0 = xs - W_SIDE + 4 * gq;
        const bool col_ok = row0 < ROWS_PER_PASS && px0 >= 0 && (size_t)px0 * 3 + 12 <= a.prev_pitch;
        const uint8_t* src = a.prev + (size_t)s * a.prev_stream + (size_t)px0 * 3;       // px0 * 3 is a multiple of 12
        uint32_t* dst = win + row0 * W_PITCH + 4 * gq;
        uint32_t pa[PASSES], pb[PASSES], pc[PASSES];
#pragma unroll
        for (int k = 0; k < PASSES; ++k) {                         // all loads first
            const int row = row0 + k * ROWS_PER_PASS, gy = yb - W_WRY + row;
            pa[k] = pb[k] = pc[k] = 0;
            if (col_ok && row < W_ROWS && gy >= 0 && gy < a.H) {
                const uint32_t* q = (const uint32_t*)(src + (size_t)gy * a.prev_pitch);
                pa[k] = __ldg(q); pb[k] = __ldg(q + 1); pc[k] = __ldg(q + 2);
            }
        }
        if (row0 < ROWS_PER_PASS) {
#pragma unroll
            for (int k = 0; k < PASSES; ++k)
                if (row0 + k * ROWS_PER_PASS < W_ROWS) store_pixels4(dst + k * ROWS_PER_PASS * W_PITCH, pa[k], pb[k], pc[k]);
        }
    }
    __syncthreads();
    const size_t g = (size_t)s * a.Gx * a.Gy + (size_t)by * a.Gx + bx;
    if (searched) {
        const WalkBounds wb = walk_bounds(a, x0, y0, 16, bh);
        const uint32_t lane_base = (uint32_t)__cvta_generic_to_shared(win) +
                                   (uint32_t)((((warp >> 3) * 16 + r + W_WRY) * W_PITCH + (x0 - xs + W_SIDE) + h) * 4);
        WalkW w = {0, 0, KIND_FIRST, 0xffffffffu, 0, 0, 0u};
        const int st = warp_walk<W_PITCH>(a, lane_base, cw, row_on, wb, w, TileReach());
        if (lane == 0) {
            if (st == 1) {
                a.mv[2 * g] = (int16_t)w.cx; a.mv[2 * g + 1] = (int16_t)w.cy; a.sse[g] = w.bs;
                if (w.bs <= a.limit[limit_index(a, 16, bh)]) {        // PSNR > T: member of Step 3's set S
                    atomicAdd(&sums[0], w.cx); atomicAdd(&sums[1], w.cy); atomicAdd(&sums[2], 1);
                }
            } else {                                                  // block, chosen next centre, its SSE, centre it was found from
                const int slot = atomicAdd(long_count, 1);
                long_list[slot] = make_uint4((uint32_t)g, tie_key(w.nx, w.ny), w.ns, (uint32_t)(w.cx + 128) | ((uint32_t)(w.cy + 128) << 8));
            }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0 && sums[2]) {                                // Step 3's sums once per CTA (one stream per CTA)
        atomicAdd(&a.acc[4 * s + 0], sums[0]);
        atomicAdd(&a.acc[4 * s + 1], sums[1]);
        atomicAdd(&a.acc[4 * s + 2], sums[2]);
    }
}

// ---------------------------------------------------------------------------------------------
// Step 2 for 16-pixel blocks, three step search (Section 7.5), several blocks per warp
// ---------------------------------------------------------------------------------------------
// Same lane layout as the diamond kernel.  Every block scores the same number of points (the centre, then
// eight per step), so the blocks of a warp stay in step without loss.  WalkState: phase = current step size,
// mask = points of the 3 x 3 grid still to score (bit 4 = its centre).
template <int LPB, typename Win>
__device__ __forceinline__ void lockstep_tss(const MatchArgs& a, const RowCtx<16 / LPB>& rc, const Win& win, int q,
                                             int dx_lo, unsigned dx_span, int dy_lo, unsigned dy_span, WalkState& w)
{
    constexpr int NR = 16 / LPB;
#pragma unroll 1
    for (int pass = 0; pass < 9 * 8; ++pass) {                   // at most 1 + 8 * log2(2 S0) points, S0 <= 64
        if (w.st == 0 && w.mask == 0) {
            w.phase >>= 1;                                        // next, halved step around the best point so far
            if (w.phase == 0) w.st = 1;
            else { w.cx = (int)(w.bt & 0xff) - 128; w.cy = (int)((w.bt >> 8) & 0xff) - 128; w.mask = 0x1efu; }
        }
        if (!__any_sync(0xffffffffu, w.st == 0)) break;
        const bool run = w.st == 0;
        const int i = run ? __ffs(w.mask) - 1 : 4;
        w.mask &= w.mask - 1;
        const int dx = w.cx + (i % 3 - 1) * w.phase, dy = w.cy + (i / 3 - 1) * w.phase;
        const bool ok = run && (unsigned)(dx - dx_lo) <= dx_span && (unsigned)(dy - dy_lo) <= dy_span;
        uint32_t ks = 0;
        if (ok) {
            uint32_t sh;
#pragma unroll
            for (int k = 0; k < NR; ++k) {
                const uint32_t* p = win.row(q + k * LPB, dx, dy, sh);
                const uint32_t v = rc.template sse<false>(k, p, sh);
                ks += rc.row_on[k] ? v : 0u;
            }
        }
#pragma unroll
        for (int off = LPB / 2; off > 0; off >>= 1) ks += __shfl_xor_sync(0xffffffffu, ks, off);
        const uint32_t kt = ((uint32_t)(abs(dx) + abs(dy)) << 16) | ((uint32_t)(dy + 128) << 8) | (uint32_t)(dx + 128);
        if (ok && (ks < w.bs || (ks == w.bs && kt < w.bt))) { w.bs = ks; w.bt = kt; }
    }
}

// Window of a CTA's 8 x VS blocks whose reach is known at launch only (three step search: 2 S0 - 1 pixels).
struct StackWinR {
    const uint32_t* win; int x0, wx0, row0, wr, pitch;
    __device__ __forceinline__ const uint32_t* row(int r, int dx, int dy, uint32_t& sh) const
    {
        const int off = (x0 + dx) * 3 - wx0;
        sh = (off & 3) * 8;
        return win + (row0 + r + dy + wr) * pitch + (off >> 2);
    }
};

// One CTA per 8 x VS blocks; the window (dynamic shared memory) reaches wr = 2 S0 - 1 pixels around the tile, which
// covers every point the search can visit.  Blocks clipped in width are left to the generic kernel.
template <int LPB, int VS>
__global__ void __launch_bounds__(LPB * 8 * VS) k_search_tss16q(MatchArgs a, int s0, int wr, int words, int pitch)
{
    extern __shared__ uint32_t tss_win[];
    constexpr int THREADS = LPB * 8 * VS;
    const int rows = 16 * VS + 2 * wr, cpr = words / 4, chunks = rows * cpr;
    const int strips = (a.Gx + 7) >> 3, vgroups = (a.Gy + VS - 1) / VS;
    const int strip = blockIdx.x % strips, vg = (blockIdx.x / strips) % vgroups, s = blockIdx.x / (strips * vgroups);
    const int xs = strip * 128, yb = vg * 16 * VS;
    const int wx0 = ((xs - wr) * 3) & ~15;                    // byte column of the window origin (may be < 0)
    const int lane = threadIdx.x & 31, q = lane % LPB;
    const int blk = threadIdx.x / LPB, by = vg * VS + (blk >> 3), bx = strip * 8 + (blk & 7);
    const bool in_grid = bx < a.Gx && by < a.Gy;
    const int x0 = bx * 16, y0 = by * 16;
    const bool searched = in_grid && a.W - x0 >= 16;
    const int bw = searched ? 16 : 0, bh = searched ? min(16, a.H - y0) : 0;
    RowCtx<16 / LPB> rc;                                      // issued first: in flight while the window is staged
    rc.load_block(a.cur + (size_t)s * a.cur_stream + (size_t)(searched ? y0 : 0) * a.cur_pitch + (size_t)(searched ? x0 : 0) * 3,
                  a.cur_pitch, q, LPB, bw, bh);
    const uint8_t* prev = a.prev + (size_t)s * a.prev_stream;
    constexpr int UNR = 4;                                    // 16-byte chunks; wx0 and the pitch are 16-byte multiples
    for (int i0 = threadIdx.x; i0 < chunks; i0 += THREADS * UNR) {
        uint4 v[UNR];
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            const int i = i0 + u * THREADS, row = i / cpr, ci = i - row * cpr;
            const int gy = yb - wr + row, gb = wx0 + ci * 16;
            v[u] = make_uint4(0, 0, 0, 0);
            if (i < chunks && gy >= 0 && gy < a.H && gb >= 0 && gb + 16 <= (int)a.prev_pitch)
                v[u] = __ldg((const uint4*)(prev + (size_t)gy * a.prev_pitch + gb));
        }
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            const int i = i0 + u * THREADS, row = i / cpr, ci = i - row * cpr;
            if (i < chunks) {
                uint32_t* d = tss_win + row * pitch + ci * 4;
                d[0] = v[u].x; d[1] = v[u].y; d[2] = v[u].z; d[3] = v[u].w;
            }
        }
    }
    __syncthreads();
    const size_t g = (size_t)s * a.Gx * a.Gy + (size_t)by * a.Gx + bx;
    const int dx_lo = max(-a.R, -x0), dy_lo = max(-a.R, -y0);
    const unsigned dx_span = (unsigned)(min(a.R, a.W - bw - x0) - dx_lo), dy_span = (unsigned)(min(a.R, a.H - bh - y0) - dy_lo);
    const StackWinR sw = {tss_win, x0, wx0, (blk >> 3) * 16, wr, pitch};
    WalkState w;
    walk_begin(w, searched);
    w.phase = s0;                                             // first pass: the centre and its eight neighbours at step S0
    if (searched && s0 == 0) w.mask = 0x010u;                 // range 0: the zero vector alone
    lockstep_tss<LPB>(a, rc, sw, q, dx_lo, dx_span, dy_lo, dy_span, w);
    const int fx = (int)(w.bt & 0xff) - 128, fy = (int)((w.bt >> 8) & 0xff) - 128;
    const bool fin = searched && q == 0;
    if (fin) { a.mv[2 * g] = (int16_t)fx; a.mv[2 * g + 1] = (int16_t)fy; a.sse[g] = w.bs; }
    const bool pass = fin && w.bs <= a.limit[limit_index(a, bw, bh)];     // PSNR > T: member of Step 3's set S
    const int n_pass = __popc(__ballot_sync(0xffffffffu, pass));
    const int sum_x = __reduce_add_sync(0xffffffffu, pass ? fx : 0), sum_y = __reduce_add_sync(0xffffffffu, pass ? fy : 0);
    if (lane == 0 && n_pass) {
        atomicAdd(&a.acc[4 * s + 0], sum_x);
        atomicAdd(&a.acc[4 * s + 1], sum_y);
        atomicAdd(&a.acc[4 * s + 2], n_pass);
    }
}

constexpr int TSS_LPB = 4, TSS_VS = 4;
// shared memory of one k_search_tss16q CTA for search range R
static size_t tss_window_bytes(int R)
{
    int s0 = R < 1 ? 0 : 1;
    while (s0 > 0 && 4 * s0 - 1 <= R) s0 *= 2;
    const int wr = s0 > 0 ? 2 * s0 - 1 : 1;
    const int words = ((((112 + 2 * wr) * 3 + 15) >> 2) + 13 + 3) & ~3;
    return (size_t)(16 * TSS_VS + 2 * wr) * (words | 1) * sizeof(uint32_t);
}

// Section 4, k-skip: blocks that are not searched report vector (0, 0) and SSE 2^32 - 1.  One thread per block.
__global__ void k_mark_unsearched(MatchArgs a)
{
    const int gi = blockIdx.x * blockDim.x + threadIdx.x;
    if (gi >= a.S * a.Gx * a.Gy) return;
    const int b = gi % (a.Gx * a.Gy), by = b / a.Gx, bx = b - by * a.Gx;
    if (bx % a.skip_k != 0 || by % a.skip_k != 0) { a.mv[2 * gi] = 0; a.mv[2 * gi + 1] = 0; a.sse[gi] = 0xffffffffu; }
}

// Phase 2: the walks that left their tile's window.  A warp takes walks off the list one after the other (atomic
// cursor); the walk gets a private window of P_ROWS x P_COLS pixels around its centre, re-staged around the next
// centre whenever that is out of reach.  A continued walk makes exactly the move it had chosen (new points only),
// so the sequence of scored candidates is the uninterrupted walk's.
// With k-skip (Section 4) the searched blocks lie k blocks apart and share no window: there is no phase 1 then,
// and this kernel walks every searched full-width block from its start (long_list == nullptr; item i is the
// i-th searched block in stream / row / column order).
constexpr int P_WARPS = 8;
constexpr int P_REACH = 8;                                  // staged pixels above and left of the block at the window's centre
constexpr int P_ROWS = 16 + 2 * P_REACH, P_COLS = 36, P_PITCH = 38;
static_assert(P_PITCH % 4 == 2 && P_PITCH >= P_COLS && P_COLS % 4 == 0 && P_COLS >= 16 + 2 * P_REACH + 3, "window of a walk");

struct PrivateReach {
    int wcx, wcy;
    __device__ __forceinline__ bool operator()(int cx, int cy) const { return abs(cx - wcx) + 2 <= P_REACH && abs(cy - wcy) + 2 <= P_REACH; }
};

__global__ void __launch_bounds__(P_WARPS * 32, 5) k_search_dsw_long(MatchArgs a, const uint4* long_list, const int32_t* long_count, int32_t* cursor)
{
    __shared__ __align__(16) uint32_t win_all[P_WARPS][P_ROWS * P_PITCH];
    const int lane = threadIdx.x & 31, r = lane >> 1, h = lane & 1;
    uint32_t* win = win_all[threadIdx.x >> 5];
    const int per = a.Gx * a.Gy;
    const bool direct = long_list == nullptr;
    const int sgx = (a.W / 16 + a.skip_k - 1) / a.skip_k, sgy = (a.Gy + a.skip_k - 1) / a.skip_k;   // searched columns (full width only), rows
    const int n = direct ? a.S * sgx * sgy : *long_count;
    const int max_rounds = 4 * a.R + 8;                               // each re-staging moves the centre by more than 4 px
#pragma unroll 1
    for (;;) {
        int idx = 0;
        if (lane == 0) idx = atomicAdd(cursor, 1);
        idx = __shfl_sync(0xffffffffu, idx, 0);
        if (idx >= n) break;
        size_t g;
        WalkW w = {0, 0, KIND_FIRST, 0xffffffffu, 0, 0, 0u};
        if (direct) {
            const int ss = idx / (sgx * sgy), q = idx - ss * sgx * sgy, sby = q / sgx, sbx = q - sby * sgx;
            g = (size_t)ss * per + (size_t)(sby * a.skip_k) * a.Gx + sbx * a.skip_k;
        } else {
            const uint4 e = long_list[idx];
            g = e.x; w.bs = e.z;
            const int ox = (int)(e.w & 0xff) - 128, oy = (int)((e.w >> 8) & 0xff) - 128;      // the centre the walk stopped at
            w.cx = (int)(e.y & 0xff) - 128; w.cy = (int)((e.y >> 8) & 0xff) - 128;            // the move it had chosen: make it
            w.kind = c_kind_of_move[((w.cy - oy + 2) * 5 + (w.cx - ox + 2)) >> 1];
        }
        const int s = (int)(g / per), b = (int)(g - (size_t)s * per), by = b / a.Gx, bx = b - by * a.Gx;
        const int x0 = bx * 16, y0 = by * 16, bh = min(16, a.H - y0);
        const bool row_on = r < bh;
        uint32_t cw[8];
        load_lane_pixels(a.cur + (size_t)s * a.cur_stream + (size_t)(row_on ? y0 + r : y0) * a.cur_pitch + (size_t)x0 * 3, h, row_on, cw);
        const uint8_t* prev = a.prev + (size_t)s * a.prev_stream;
        const WalkBounds wb = walk_bounds(a, x0, y0, 16, bh);
#pragma unroll 1
        for (int round = 0;; ++round) {
            // the window around the centre that is scored next
            const PrivateReach reach = {w.cx, w.cy};
            const int wx0 = (x0 + w.cx - P_REACH) & ~3, wy0 = y0 + w.cy - P_REACH;
            {   // a lane keeps its group of 4 pixels (one column position) and goes down the rows, 3 rows apart
                constexpr int GROUPS = P_COLS / 4, RPP = 32 / GROUPS, PASSES = (P_ROWS + RPP - 1) / RPP, HALF = (PASSES + 1) / 2;
                const int gq = lane % GROUPS, row0 = lane / GROUPS, px0 = wx0 + 4 * gq;
                const bool col_ok = row0 < RPP && px0 >= 0 && (size_t)px0 * 3 + 12 <= a.prev_pitch;
                const uint8_t* src = prev + (size_t)px0 * 3;                          // px0 * 3 is a multiple of 12
                uint32_t* dst = win + row0 * P_PITCH + 4 * gq;
#pragma unroll
                for (int half = 0; half < 2; ++half) {                               // loads of half the passes, then their stores
                    uint32_t pa[HALF], pb[HALF], pc[HALF];
#pragma unroll
                    for (int k = 0; k < HALF; ++k) {
                        const int row = row0 + (half * HALF + k) * RPP, gy = wy0 + row;
                        pa[k] = pb[k] = pc[k] = 0;
                        if (col_ok && row < P_ROWS && gy >= 0 && gy < a.H) {
                            const uint32_t* q = (const uint32_t*)(src + (size_t)gy * a.prev_pitch);
                            pa[k] = __ldg(q); pb[k] = __ldg(q + 1); pc[k] = __ldg(q + 2);
                        }
                    }
#pragma unroll
                    for (int k = 0; k < HALF; ++k) {
                        const int row = row0 + (half * HALF + k) * RPP;
                        if (row0 < RPP && row < P_ROWS) store_pixels4(dst + (half * HALF + k) * RPP * P_PITCH, pa[k], pb[k], pc[k]);
                    }
                }
            }
            __syncwarp();
            // this lane's first word at displacement (0, 0): frame row y0 + r, pixel x0 + h, relative to the window's
            // origin (it may lie outside the window; only displacements near the centre are ever addressed)
            const uint32_t lane_base = (uint32_t)__cvta_generic_to_shared(win) + (uint32_t)(((r + y0 - wy0) * P_PITCH + (x0 - wx0) + h) * 4);
            const int st = warp_walk<P_PITCH>(a, lane_base, cw, row_on, wb, w, reach);
            if (st == 1) break;
            if (round >= max_rounds) {                                   // never reached; a walk cut here is not valid
                if (lane == 0) atomicExch(a.status, (int)DC_ERR_TIMEOUT);
                break;
            }
            // make the chosen move; the next round scores its new points in a window around the new centre
            w.kind = c_kind_of_move[((w.ny - w.cy + 2) * 5 + (w.nx - w.cx + 2)) >> 1];
            w.cx = w.nx; w.cy = w.ny; w.bs = w.ns;
            __syncwarp();                                                // every lane has finished reading the old window
        }
        if (lane == 0) publish_block(a, s, g, 16, bh, ((unsigned long long)w.bs << 32) | tie_key(w.cx, w.cy));
    }
}

// Step 4 for 16-pixel blocks, in two launches.
// k_verify16_prep (one thread per block) rounds M, settles every block that needs no pixels -- M leaves the frame
// or the range for it, or its own best vector is M, so that Step 2 already holds the score (Section 4's second
// acceleration, exact in that case) -- and lists the others.  k_verify16_list scores the listed blocks, one
// half-warp per block and one lane per block row, so that no warp idles on blocks that were settled.
__global__ void __launch_bounds__(256) k_verify16_prep(MatchArgs a, uint32_t* list, int32_t* list_count)
{
    const int lane = threadIdx.x & 31;
    const int per = a.Gx * a.Gy;
    const unsigned gi = blockIdx.x * 256u + threadIdx.x;                          // S * Gx * Gy < 2^31
    const bool in_grid = gi < (unsigned)(per * a.S);
    const int s = in_grid ? (int)(gi / (unsigned)per) : a.S - 1, b = in_grid ? (int)(gi - (unsigned)s * per) : 0;
    const int by = b / a.Gx, bx = b - by * a.Gx;
    const int x0 = bx * 16, y0 = by * 16, bw = min(16, a.W - x0), bh = min(16, a.H - y0);
    const int4 sums = __ldcg((const int4*)a.acc + s);                            // Step 3: sum dx, sum dy, K (one 16-byte load)
    const int K = sums.z;
    int Mx = 0, My = 0;
    if (K > 0) { Mx = round_mean(sums.x, K); My = round_mean(sums.y, K); }
    const bool cand_ok = in_grid && K > 0 && abs(Mx) <= a.R && abs(My) <= a.R && x0 + Mx >= 0 && y0 + My >= 0 &&
                         x0 + Mx + bw <= a.W && y0 + My + bh <= a.H;
    bool known = false; uint32_t v = 0;
    if (cand_ok) {
        const uint32_t own = ((const uint32_t*)a.mv)[gi];                         // (dx, dy) as one word
        v = a.sse[gi];
        known = (int16_t)(own & 0xffffu) == Mx && (int16_t)(own >> 16) == My && v != 0xffffffffu;
    }
    const bool settled = in_grid && (!cand_ok || known);
    const int ok = known && v <= a.limit[limit_index(a, bw, bh)];
    if (settled) a.matched[gi] = (uint8_t)ok;
    if (in_grid && b == 0) { a.gmv[3 * s] = Mx; a.gmv[3 * s + 1] = My; a.gmv[3 * s + 2] = K; }
    // matched count: one atomic per warp and stream
    const unsigned same = __match_any_sync(0xffffffffu, s);
    const unsigned oks = __ballot_sync(0xffffffffu, ok);
    if (lane == __ffs(same) - 1 && (oks & same)) atomicAdd(&a.acc[4 * s + 3], __popc(oks & same));
    // the blocks whose pixels must be read
    const bool todo = in_grid && !settled;
    const unsigned tm = __ballot_sync(0xffffffffu, todo);
    if (tm) {
        int base = 0;
        if (lane == 0) base = atomicAdd(list_count, __popc(tm));
        base = __shfl_sync(0xffffffffu, base, 0);
        if (todo) list[base + __popc(tm & ((1u << lane) - 1u))] = gi;
    }
}

__global__ void __launch_bounds__(256) k_verify16_list(MatchArgs a, const uint32_t* list, const int32_t* list_count)
{
    const int lane = threadIdx.x & 31, r = lane & 15, half = lane >> 4;
    const int per = a.Gx * a.Gy, n = *list_count;
    const int stride = gridDim.x * 16;
    for (int i0 = (blockIdx.x * 8 + (threadIdx.x >> 5)) * 2; i0 < n; i0 += stride) {      // both halves of a warp stay in the loop together
        const int i = i0 + half;
        const bool on = i < n;
        const unsigned gi = on ? list[i] : 0u;
        const int s = (int)(gi / (unsigned)per), b = (int)(gi - (unsigned)s * per);
        const int by = b / a.Gx, bx = b - by * a.Gx;
        const int x0 = bx * 16, y0 = by * 16, bw = min(16, a.W - x0), bh = min(16, a.H - y0);
        const int Mx = a.gmv[3 * s], My = a.gmv[3 * s + 1];
        uint32_t acc = 0;
        if (on && r < bh) {
            RowCtx<1> rc;
            rc.load_block(a.cur + (size_t)s * a.cur_stream + (size_t)y0 * a.cur_pitch + (size_t)x0 * 3, a.cur_pitch, r, 16, bw, bh);
            // the 48 bytes of the displaced row lie in four aligned 16-byte chunks (rows of the frame copy are padded):
            // four wide loads instead of thirteen narrow ones, then a word offset that is the same for a whole stream
            const uint8_t* p = a.prev + (size_t)s * a.prev_stream + (size_t)(y0 + My + r) * a.prev_pitch + (size_t)(x0 + Mx) * 3;
            const uint4* p16 = (const uint4*)((uintptr_t)p & ~(uintptr_t)15);
            const uint4 c0 = __ldg(p16), c1 = __ldg(p16 + 1), c2 = __ldg(p16 + 2), c3 = __ldg(p16 + 3);
            const uint32_t ww[16] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w, c2.x, c2.y, c2.z, c2.w, c3.x, c3.y, c3.z, c3.w};
            const uint32_t boff = (uint32_t)(uintptr_t)p & 15u, sh = (boff & 3u) * 8u;
            uint32_t w[13];
            switch (boff >> 2) {
            case 0:
#pragma unroll
                for (int j = 0; j < 13; ++j) w[j] = ww[j];
                break;
            case 1:
#pragma unroll
                for (int j = 0; j < 13; ++j) w[j] = ww[j + 1];
                break;
            case 2:
#pragma unroll
                for (int j = 0; j < 13; ++j) w[j] = ww[j + 2];
                break;
            default:
#pragma unroll
                for (int j = 0; j < 13; ++j) w[j] = ww[j + 3];
                break;
            }
            acc = rc.sse_words(0, w, sh);
        }
        const uint32_t sse = __reduce_add_sync(half ? 0xffff0000u : 0x0000ffffu, acc);
        if (r == 0 && on) {
            const int ok = sse <= a.limit[limit_index(a, bw, bh)];
            a.matched[gi] = (uint8_t)ok;
            if (ok) atomicAdd(&a.acc[4 * s + 3], 1);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Fast Step 2: 16-pixel blocks, exhaustive search (plain integer ALU work: every displacement is scored)
// ---------------------------------------------------------------------------------------------
// One CTA per strip of 8 blocks, one warp per block.  The strip's search window (16 + 2R rows) is staged in
// shared memory once.  A lane owns one horizontal displacement dx; for one 4-byte column of the block it
// keeps the 16 rows of the current block in registers and walks down the window: every previous-frame word
// it loads is scored against all block rows it can pair with, i.e. for E_DY vertical displacements at once,
// so one (unaligned) load feeds up to 16 difference/accumulate pairs.  Displacements beyond the last full
// group of 32 dx values are scored one candidate per lane.  Blocks clipped by the frame edge are left to
// the generic kernel.
constexpr int E_DY = 13;                        // vertical displacements scored together (65 = 5 * 13 for R = 32)
constexpr int E_MAXR = 32;
constexpr int E_PITCH = 152;                    // window row in words: (128 + 64) px * 3 B + 15 B alignment + one spare word, 16-byte multiple
constexpr int E_MAXROWS = 16 + 2 * E_MAXR + E_DY - 1;   // plus rows only touched by displacements beyond R (scored, never compared)

__global__ void __launch_bounds__(256, 3) k_search_es16(MatchArgs a)
{
    extern __shared__ uint32_t es_sm[];
    const int R = a.R, n_d = 2 * R + 1;
    const int chunks = (n_d + E_DY - 1) / E_DY;
    const int rows = 16 + chunks * E_DY - 1;                     // <= E_MAXROWS
    uint32_t* win = es_sm;
    uint32_t* cur_all = es_sm + rows * E_PITCH;
    const int strips = (a.Gx + 7) >> 3;
    const int strip = blockIdx.x % strips, by = (blockIdx.x / strips) % a.Gy, s = blockIdx.x / (strips * a.Gy);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int xs = strip * 128, y0 = by * 16;
    const int wx0 = ((xs - R) * 3) & ~15;                        // byte column of the window origin (may be < 0)
    const uint8_t* prev = a.prev + (size_t)s * a.prev_stream;
    const bool row_searched = (a.skip_k <= 1 || by % a.skip_k == 0) && a.H - y0 >= 16;
    for (int i = threadIdx.x; row_searched && i < rows * (E_PITCH / 4); i += 256) {
        const int row = i / (E_PITCH / 4), ci = i - row * (E_PITCH / 4);
        const int gy = y0 - R + row, gb = wx0 + ci * 16;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (gy >= 0 && gy < a.H && gb >= 0 && gb + 16 <= (int)a.prev_pitch)
            v = __ldg((const uint4*)(prev + (size_t)gy * a.prev_pitch + gb));
        *(uint4*)(win + row * E_PITCH + ci * 4) = v;
    }
    const int bx = strip * 8 + warp, x0 = bx * 16;
    const bool full = bx < a.Gx && a.W - x0 >= 16 && a.H - y0 >= 16;
    const bool skipped = a.skip_k > 1 && (bx % a.skip_k != 0 || by % a.skip_k != 0);
    uint32_t* curw = cur_all + warp * 192;
    if (full && !skipped) {                                       // the current block: 16 rows of 48 bytes
        const uint8_t* cb = a.cur + (size_t)s * a.cur_stream + (size_t)y0 * a.cur_pitch + (size_t)x0 * 3;
        for (int i = lane; i < 16 * 3; i += 32) {
            const int r = i / 3, q = i - r * 3;
            *(uint4*)(curw + r * 12 + q * 4) = __ldg((const uint4*)(cb + (size_t)r * a.cur_pitch) + q);
        }
    }
    __syncthreads();
    if (bx >= a.Gx) return;
    const size_t g = (size_t)s * a.Gx * a.Gy + (size_t)by * a.Gx + bx;
    if (skipped) {
        if (lane == 0) { a.mv[2 * g] = 0; a.mv[2 * g + 1] = 0; a.sse[g] = 0xffffffffu; }
        return;
    }
    if (!full) return;                                            // clipped block: the generic kernel scores it

    unsigned long long bk = ~0ull;
    const int full_passes = n_d / 32;
    for (int pass = 0; pass < full_passes; ++pass) {
        const int dx = -R + pass * 32 + lane;
        const int boff = (x0 + dx) * 3 - wx0;
        const uint32_t sh = (boff & 3) * 8;
        const bool x_ok = x0 + dx >= 0 && x0 + dx + 16 <= a.W;
        for (int c = 0; c < chunks; ++c) {
            const int dy0 = -R + c * E_DY;
            uint32_t acc[E_DY];
#pragma unroll
            for (int d = 0; d < E_DY; ++d) acc[d] = 0;
            const uint32_t* col = win + (c * E_DY) * E_PITCH + (boff >> 2);      // window row of displacement dy0, block row 0
#pragma unroll 1
            for (int j = 0; j < 12; ++j) {
                uint32_t cw[16];
#pragma unroll
                for (int r = 0; r < 16; ++r) cw[r] = curw[r * 12 + j];
#pragma unroll
                for (int p = 0; p < 16 + E_DY - 1; ++p) {
                    const uint32_t w = __funnelshift_r(col[p * E_PITCH + j], col[p * E_PITCH + j + 1], sh);
#pragma unroll
                    for (int r = 0; r < 16; ++r) {
                        if (p - r >= 0 && p - r < E_DY) {
                            const uint32_t t = __vabsdiffu4(cw[r], w);
                            acc[p - r] = __dp4a(t, t, acc[p - r]);
                        }
                    }
                }
            }
#pragma unroll
            for (int d = 0; d < E_DY; ++d) {
                const int dy = dy0 + d;
                if (x_ok && dy <= R && y0 + dy >= 0 && y0 + dy + 16 <= a.H) {
                    const unsigned long long k = cand_key(acc[d], dx, dy);
                    if (k < bk) bk = k;
                }
            }
        }
    }
    // the remaining dx columns: one candidate per lane and round
    const int dx_first = -R + full_passes * 32, n_left = (n_d - full_passes * 32) * n_d;
    for (int i = lane; i < n_left; i += 32) {
        const int dx = dx_first + i / n_d, dy = -R + i % n_d;
        if (x0 + dx < 0 || x0 + dx + 16 > a.W || y0 + dy < 0 || y0 + dy + 16 > a.H) continue;
        const int boff = (x0 + dx) * 3 - wx0;
        const uint32_t sh = (boff & 3) * 8;
        const uint32_t* col = win + (dy + R) * E_PITCH + (boff >> 2);
        uint32_t acc = 0;
#pragma unroll 2
        for (int r = 0; r < 16; ++r) {
            uint32_t lo = col[r * E_PITCH];
#pragma unroll
            for (int j = 0; j < 12; ++j) {
                const uint32_t hi = col[r * E_PITCH + j + 1];
                const uint32_t t = __vabsdiffu4(curw[r * 12 + j], __funnelshift_r(lo, hi, sh));
                acc = __dp4a(t, t, acc);
                lo = hi;
            }
        }
        const unsigned long long k = cand_key(acc, dx, dy);
        if (k < bk) bk = k;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(0xffffffffu, bk, o);
        if (other < bk) bk = other;
    }
    if (lane == 0) publish_block(a, s, g, 16, 16, bk);            // the zero vector is always valid, so bk is set
}

// Frame -> the library's aligned copy.  16-byte vectors when the source rows are aligned.
__global__ void k_copy_frame(const uint8_t* src, size_t src_pitch, uint8_t* dst, size_t dst_pitch, int row_bytes,
                             int rows, int vec)
{
    if (vec) {
        const int chunks = (row_bytes + 15) >> 4;             // the last chunk may read source padding? no: see below
        const size_t total = (size_t)rows * chunks;
        for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
            const size_t row = i / chunks; const int c = (int)(i - row * chunks);
            if (c * 16 + 16 <= row_bytes) {
                *(uint4*)(dst + row * dst_pitch + c * 16) = __ldg((const uint4*)(src + row * src_pitch + c * 16));
            } else {                                          // ragged tail of the row: byte by byte
                for (int k = c * 16; k < row_bytes; ++k) dst[row * dst_pitch + k] = src[row * src_pitch + k];
            }
        }
    } else {
        const size_t total = (size_t)rows * row_bytes;
        for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
            const size_t row = i / row_bytes; const int k = (int)(i - row * row_bytes);
            dst[row * dst_pitch + k] = src[row * src_pitch + k];
        }
    }
}

template <int ITERS>
void launch_generic(dc_cache* c, MatchArgs& a, bool search)
{
    int warps = a.S * a.Gx * a.Gy;
    int grid = dc_div_up(warps, WARPS);
    if (search) { dc_prof_scope ps(c, DC_ST_SEARCH); k_search<ITERS><<<grid, WARPS * 32, 0, c->stream>>>(a); }
    else { dc_prof_scope ps(c, DC_ST_VERIFY); k_verify<ITERS><<<grid, WARPS * 32, 0, c->stream>>>(a); }
}

void launch_by_block(dc_cache* c, MatchArgs& a, bool search)
{
    int row_words = (a.B * 3 + 3) / 4, iters = dc_div_up(a.B * row_words, 32);
    if (iters <= 2) launch_generic<2>(c, a, search);
    else if (iters <= 3) launch_generic<3>(c, a, search);
    else if (iters <= 6) launch_generic<6>(c, a, search);
    else if (iters <= 12) launch_generic<12>(c, a, search);
    else launch_generic<24>(c, a, search);
}

}  // namespace

int dc_launch_copy_frame(dc_cache* c, const uint8_t* frame, size_t pitch, uint8_t* dst)
{
    const int row_bytes = c->cfg.width * 3, rows = c->cfg.height * c->S;
    const int vec = ((uintptr_t)frame % 16 == 0) && (pitch % 16 == 0);
    size_t work = vec ? (size_t)rows * ((row_bytes + 15) / 16) : (size_t)rows * row_bytes;
    int grid = (int)((work + 255) / 256);
    if (grid > c->num_sms * 16) grid = c->num_sms * 16;
    if (grid < 1) grid = 1;
    dc_prof_scope ps(c, DC_ST_KEY_UPDATE);
    k_copy_frame<<<grid, 256, 0, c->stream>>>(frame, pitch, dst, c->key_pitch, row_bytes, rows, vec);
    c->launches += 1;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}

int dc_launch_match(dc_cache* c, const uint8_t* cur_key, const uint8_t* prev_key)
{
    MatchArgs a;
    a.cur = cur_key; a.cur_pitch = c->key_pitch; a.cur_stream = c->key_pitch * (size_t)c->cfg.height;
    a.prev = prev_key; a.prev_pitch = c->key_pitch; a.prev_stream = c->key_pitch * (size_t)c->cfg.height;
    a.W = c->cfg.width; a.H = c->cfg.height; a.B = c->cfg.block; a.R = c->cfg.range;
    a.Gx = c->Gx; a.Gy = c->Gy; a.S = c->S; a.search = c->cfg.search; a.skip_k = c->cfg.skip_k; a.region_mode = c->cfg.region_mode; a.edge_only = 0;
    for (int i = 0; i < 4; ++i) a.limit[i] = c->sse_limit[i];
    a.mv = c->blk_mv; a.sse = c->blk_sse; a.matched = c->matched; a.acc = c->mv_acc; a.gmv = c->gmv;
    a.status = c->status;
    // Step 3 sums and, behind them, the counter of walks handed to the second search phase
    DC_CUDA(cudaMemsetAsync(c->mv_acc, 0, sizeof(int32_t) * (4 * c->S + 4), c->stream));
    int32_t* long_count = c->mv_acc + 4 * c->S;
    if (a.B == 16 && a.search == DC_SEARCH_DIAMOND) {
        {
            dc_prof_scope ps(c, DC_ST_SEARCH);
            if (a.skip_k <= 1) {
                const dim3 tiles((a.Gx + 7) / 8, (a.Gy + W_VS - 1) / W_VS, a.S);
                k_search_dsw<<<tiles, W_VS * 8 * 32, 0, c->stream>>>(a, c->long_list, long_count);
                k_search_dsw_long<<<c->num_sms * 5, P_WARPS * 32, 0, c->stream>>>(a, c->long_list, long_count, long_count + 1);
            } else {
                k_mark_unsearched<<<dc_div_up(a.S * a.Gx * a.Gy, 256), 256, 0, c->stream>>>(a);
                k_search_dsw_long<<<c->num_sms * 5, P_WARPS * 32, 0, c->stream>>>(a, nullptr, long_count, long_count + 1);
            }
            c->launches += 1;
        }
        if (a.W % 16 != 0) {                                        // blocks clipped by the right edge
            a.edge_only = 2;
            launch_by_block(c, a, true);
            a.edge_only = 0;
            c->launches += 1;
        }
    } else if (a.B == 16 && a.search == DC_SEARCH_THREE_STEP && a.skip_k <= 1 && tss_window_bytes(a.R) <= 160 * 1024) {
        int s0 = a.R < 1 ? 0 : 1;                                   // first step: the largest power of two with 2 S0 - 1 <= R
        while (s0 > 0 && 4 * s0 - 1 <= a.R) s0 *= 2;
        const int wr = s0 > 0 ? 2 * s0 - 1 : 1;
        const int words = ((((112 + 2 * wr) * 3 + 15) >> 2) + 13 + 3) & ~3, pitch = words | 1;
        const size_t smem = tss_window_bytes(a.R);
        static dc_once_per_device attr_set;
        if (attr_set.first(c->device)) {
            DC_CUDA(cudaFuncSetAttribute(k_search_tss16q<TSS_LPB, TSS_VS>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024));
        }
        {
            dc_prof_scope ps(c, DC_ST_SEARCH);
            const int ctas = ((a.Gx + 7) / 8) * ((a.Gy + TSS_VS - 1) / TSS_VS) * a.S;
            k_search_tss16q<TSS_LPB, TSS_VS><<<ctas, TSS_LPB * 8 * TSS_VS, smem, c->stream>>>(a, s0, wr, words, pitch);
        }
        if (a.W % 16 != 0) {                                        // blocks clipped by the right edge
            a.edge_only = 2;
            launch_by_block(c, a, true);
            a.edge_only = 0;
            c->launches += 1;
        }
    } else if (a.B == 16 && a.search == DC_SEARCH_EXHAUSTIVE && a.R <= E_MAXR && a.W >= 16 && a.H >= 16) {
        const int chunks = (2 * a.R + 1 + E_DY - 1) / E_DY;
        const size_t smem = ((size_t)(16 + chunks * E_DY - 1) * E_PITCH + 8 * 192) * sizeof(uint32_t);
        static dc_once_per_device attr_set;
        if (attr_set.first(c->device)) {
            DC_CUDA(cudaFuncSetAttribute(k_search_es16, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)(((size_t)E_MAXROWS * E_PITCH + 8 * 192) * sizeof(uint32_t))));
        }
        {
            dc_prof_scope ps(c, DC_ST_SEARCH);
            k_search_es16<<<((a.Gx + 7) / 8) * a.Gy * a.S, 256, smem, c->stream>>>(a);
        }
        if (a.W % 16 != 0 || a.H % 16 != 0) {                   // blocks clipped by the right / bottom edge
            a.edge_only = 1;
            launch_by_block(c, a, true);
            a.edge_only = 0;
            c->launches += 1;
        }
    } else {
        launch_by_block(c, a, true);
    }
    if (a.region_mode == DC_REGIONS_PER_BLOCK) {
        dc_prof_scope ps(c, DC_ST_VERIFY);
        k_accept_own<<<dc_div_up(a.S * a.Gx * a.Gy, 256), 256, 0, c->stream>>>(a);
    } else if (a.B == 16) {
        dc_prof_scope ps(c, DC_ST_VERIFY);
        int32_t* todo_count = long_count + 2;                       // zeroed with the Step 3 sums; the walk list is free again
        k_verify16_prep<<<dc_div_up(a.S * a.Gx * a.Gy, 256), 256, 0, c->stream>>>(a, (uint32_t*)c->long_list, todo_count);
        k_verify16_list<<<c->num_sms * 8, 256, 0, c->stream>>>(a, (const uint32_t*)c->long_list, todo_count);
        c->launches += 1;
    } else {
        launch_by_block(c, a, false);
    }
    {
        dc_prof_scope ps(c, DC_ST_MERGE);
        const int16_t* own = a.region_mode == DC_REGIONS_PER_BLOCK ? c->blk_mv : nullptr;
        k_merge_runs<<<dc_div_up(c->S * a.Gx * a.Gy, 256), 256, 0, c->stream>>>(c->matched, own, a.Gx, c->S * a.Gx * a.Gy, c->run_end);
        k_merge<<<c->S, 1024, 0, c->stream>>>(c->run_end, own, c->gmv, a.W, a.H, a.B, a.Gx, a.Gy, c->max_regions,
                                              c->regions0, c->n_regions, c->status);
    }
    c->launches += 4;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}
