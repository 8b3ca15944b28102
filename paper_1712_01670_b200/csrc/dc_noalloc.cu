// dc_search_blocks_noalloc: block search (Section 4, Steps 2 and 3) for callers that cannot
// allocate device memory.
//
// The regular matcher keeps its Step 3 accumulators (sum of motion vectors and count of blocks
// that pass the PSNR test, per stream) in memory that dc_cache_create allocates.  Some callers
// have no chance to create a cache: code that runs where cudaMalloc is off limits (for instance
// a latency-critical loop whose memory was fixed at start-up), or a plug-in whose host forbids
// allocation after initialisation.  This entry point does the same
// search with the accumulators in a fixed array that lives in the library image itself.
//
// The array holds DC_NOALLOC_MAX_STREAMS x 4 32-bit words (1 KiB).  Every GPU that loads the
// library holds its own copy until the process exits.  All calls on a device share it: each
// call clears the words it uses before its kernels run, and two calls that overlap on the GPU
// (different streams, no ordering between them) race on it and give wrong motion sums.
#include <math.h>

#include "dc_common.cuh"

namespace {

constexpr int kMaxDevices = 64;
constexpr int kWarps = 8;
constexpr int kMaxRowWords = 24;              // blocks up to 32 px: 96 bytes per row

// Step 3 accumulators: per stream sum dx, sum dy, K, unused
static __device__ __align__(256) int32_t g_noalloc_acc[4 * DC_NOALLOC_MAX_STREAMS];

struct NaArgs {
    const uint8_t* cur; const uint8_t* prev; size_t pitch, stream_bytes;
    int W, H, B, R, Gx, Gy, S, search;
    uint32_t limit[4];
    int16_t* mv; uint32_t* sse; int32_t* gmv; int32_t* acc;
};

__device__ __forceinline__ unsigned long long na_key(uint32_t sse, int dx, int dy)
{
    return ((unsigned long long)sse << 32) | ((unsigned long long)(abs(dx) + abs(dy)) << 16) |
           ((unsigned long long)(dy + 128) << 8) | (unsigned long long)(dx + 128);
}

// One warp per block.  Both frames are the caller's memory with no padding promise, so every
// pixel is fetched with byte loads that stay inside the rows: slower than the cache's matcher,
// which owns padded copies of the frames, but safe for any pitch and alignment.
__global__ void __launch_bounds__(kWarps * 32) k_search_noalloc(NaArgs a)
{
    __shared__ uint32_t cur_sm[kWarps][32 * kMaxRowWords];
    const int warp = blockIdx.x * kWarps + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    const int per = a.Gx * a.Gy;
    if (warp >= per * a.S) return;
    const int s = warp / per, b = warp - s * per, by = b / a.Gx, bx = b - by * a.Gx;
    const int x0 = bx * a.B, y0 = by * a.B, bw = min(a.B, a.W - x0), bh = min(a.B, a.H - y0);
    const int row_bytes = bw * 3, wpr = (row_bytes + 3) >> 2, items = bh * wpr;
    const uint8_t* cur = a.cur + (size_t)s * a.stream_bytes;
    const uint8_t* prev = a.prev + (size_t)s * a.stream_bytes;
    uint32_t* sm = cur_sm[threadIdx.x >> 5];
    auto load_word = [&](const uint8_t* row, int wi) {     // 4 bytes of a row, zero past its end
        uint32_t v = 0;
        for (int k = 0; k < 4; ++k)
            if (wi * 4 + k < row_bytes) v |= (uint32_t)__ldg(row + wi * 4 + k) << (8 * k);
        return v;
    };
    for (int item = lane; item < items; item += 32) {
        const int row = item / wpr, wi = item - row * wpr;
        sm[row * kMaxRowWords + wi] = load_word(cur + (size_t)(y0 + row) * a.pitch + (size_t)x0 * 3, wi);
    }
    __syncwarp();
    auto valid = [&](int dx, int dy) {
        return abs(dx) <= a.R && abs(dy) <= a.R && x0 + dx >= 0 && y0 + dy >= 0 && x0 + dx + bw <= a.W && y0 + dy + bh <= a.H;
    };
    auto sse_at = [&](int dx, int dy) {
        uint32_t acc = 0;
        for (int item = lane; item < items; item += 32) {
            const int row = item / wpr, wi = item - row * wpr;
            const uint32_t pv = load_word(prev + (size_t)(y0 + dy + row) * a.pitch + (size_t)(x0 + dx) * 3, wi);
            const uint32_t d = __vabsdiffu4(sm[row * kMaxRowWords + wi], pv);
            acc = __dp4a(d, d, acc);
        }
        return __reduce_add_sync(0xffffffffu, acc);
    };
    int bdx = 0, bdy = 0;
    uint32_t bs = sse_at(0, 0);
    unsigned long long bk = na_key(bs, 0, 0);
    auto consider = [&](int dx, int dy) {
        if (!valid(dx, dy)) return;
        const uint32_t v = sse_at(dx, dy);
        const unsigned long long k = na_key(v, dx, dy);
        if (k < bk) { bk = k; bs = v; bdx = dx; bdy = dy; }
    };
    if (a.search == DC_SEARCH_EXHAUSTIVE) {
        for (int dy = -a.R; dy <= a.R; ++dy)
            for (int dx = -a.R; dx <= a.R; ++dx)
                if (dx != 0 || dy != 0) consider(dx, dy);
    } else {
        const int max_steps = (2 * a.R + 1) * (2 * a.R + 1);
        for (int step = 0; step < max_steps; ++step) {
            const int cx = bdx, cy = bdy;
            consider(cx, cy - 2); consider(cx - 1, cy - 1); consider(cx + 1, cy - 1); consider(cx - 2, cy);
            consider(cx + 2, cy); consider(cx - 1, cy + 1); consider(cx + 1, cy + 1); consider(cx, cy + 2);
            if (bdx == cx && bdy == cy) break;
        }
        const int cx = bdx, cy = bdy;
        consider(cx, cy - 1); consider(cx - 1, cy); consider(cx + 1, cy); consider(cx, cy + 1);
    }
    if (lane == 0) {
        const size_t g = (size_t)s * per + b;
        a.mv[2 * g] = (int16_t)bdx; a.mv[2 * g + 1] = (int16_t)bdy; a.sse[g] = bs;
        if (bs <= a.limit[(bh < a.B ? 2 : 0) + (bw < a.B ? 1 : 0)]) {
            atomicAdd(&a.acc[4 * s + 0], bdx);
            atomicAdd(&a.acc[4 * s + 1], bdy);
            atomicAdd(&a.acc[4 * s + 2], 1);
        }
    }
}

// Step 3: mean vector, rounded to nearest with halves away from zero
__global__ void k_mean_noalloc(const int32_t* acc, int S, int32_t* gmv)
{
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= S) return;
    const int sx = acc[4 * s], sy = acc[4 * s + 1], K = acc[4 * s + 2];
    int mx = 0, my = 0;
    if (K > 0) {
        mx = (2 * abs(sx) + K) / (2 * K); if (sx < 0) mx = -mx;
        my = (2 * abs(sy) + K) / (2 * K); if (sy < 0) my = -my;
    }
    gmv[3 * s] = mx; gmv[3 * s + 1] = my; gmv[3 * s + 2] = K;
}

// Device address of the scratch array, looked up once per device (the symbol's name is only a
// host-side handle; kernels need the address cudaGetSymbolAddress returns for the current device).
int32_t* g_scratch_ptr[kMaxDevices];

}  // namespace

extern "C" int dc_search_blocks_noalloc(const uint8_t* frame_dev, const uint8_t* prev_dev, size_t pitch_bytes,
                                        int32_t width, int32_t height, int32_t n_streams, int32_t block, int32_t range,
                                        int32_t search, double psnr_db, int16_t* block_mv_dev, uint32_t* block_sse_dev,
                                        int32_t* global_mv_dev, void* cuda_stream)
{
    if (!frame_dev || !prev_dev || !block_mv_dev || !block_sse_dev || !global_mv_dev) return DC_ERR_ARG;
    if (width < 1 || height < 1 || n_streams < 1 || pitch_bytes < (size_t)width * 3) return DC_ERR_ARG;
    if (block < 4 || block > 32 || range < 0 || range > 64) return DC_ERR_CONFIG;
    if (search != DC_SEARCH_EXHAUSTIVE && search != DC_SEARCH_DIAMOND) return DC_ERR_CONFIG;
    if (!(psnr_db > 0.0) || !(psnr_db < 200.0)) return DC_ERR_CONFIG;
    if (n_streams > DC_NOALLOC_MAX_STREAMS) return DC_ERR_LIMIT;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    int dev = 0;
    DC_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return DC_ERR_LIMIT;
    if (!g_scratch_ptr[dev]) {               // first call on this device: resolve the symbol
        int32_t* p = nullptr;
        DC_CUDA(cudaGetSymbolAddress((void**)&p, g_noalloc_acc));
        g_scratch_ptr[dev] = p;
    }
    NaArgs a;
    a.cur = frame_dev; a.prev = prev_dev; a.pitch = pitch_bytes; a.stream_bytes = pitch_bytes * (size_t)height;
    a.W = width; a.H = height; a.B = block; a.R = range; a.S = n_streams; a.search = search;
    a.Gx = dc_div_up(width, block); a.Gy = dc_div_up(height, block);
    for (int i = 0; i < 4; ++i) {
        const int bw = (i & 1) ? width - (a.Gx - 1) * block : block, bh = (i & 2) ? height - (a.Gy - 1) * block : block;
        const double lim = ceil(65025.0 * (double)(bw * bh * 3) / pow(10.0, psnr_db / 10.0)) - 1.0;
        a.limit[i] = lim >= 4294967295.0 ? 4294967295u : (uint32_t)lim;
    }
    a.mv = block_mv_dev; a.sse = block_sse_dev; a.gmv = global_mv_dev; a.acc = g_scratch_ptr[dev];
    // the array keeps the previous call's sums: clear this call's part first
    DC_CUDA(cudaMemsetAsync(a.acc, 0, sizeof(int32_t) * 4 * n_streams, stream));
    const long long warps = (long long)n_streams * a.Gx * a.Gy;
    k_search_noalloc<<<(unsigned)((warps + kWarps - 1) / kWarps), kWarps * 32, 0, stream>>>(a);
    k_mean_noalloc<<<dc_div_up(n_streams, 64), 64, 0, stream>>>(a.acc, n_streams, global_mv_dev);
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}
