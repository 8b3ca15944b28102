// Region propagation (Section 5, Table 2) and the reuse step of the cache-aware convolution
// (Section 5, "Reuse": copy cached regions, build the bitmap, list what is left to compute).
//
//   k_propagate      one thread per (stream, rectangle slot) walks the layer table in order and
//                    writes the rectangle's image after every layer.  Slots are independent,
//                    so no synchronisation is needed; a vanished rectangle is all zeros.
//   k_classify_copy  one warp per 16x8 output tile: lanes test the stream's rectangles against
//                    the tile, OR their coverage into a 128-bit bitmap, the warp copies each
//                    covered span from the cached map with 16-byte vectors, and tiles that
//                    still hold uncovered pixels are appended to the layer's dirty list.
#include "dc_common.cuh"

namespace {

__device__ __forceinline__ int floor_div(int a, int b)
{
    int q = a / b, r = a - q * b;
    return (r != 0 && ((r < 0) != (b < 0))) ? q - 1 : q;
}
__device__ __forceinline__ int ceil_div(int a, int b) { return -floor_div(-a, b); }

// Sliding window on one axis: output o reads [o s - p, o s - p + k - 1]; reusable iff that lies
// inside [x, x + w).  First = ceil((x + p) / s) as printed in Table 2; last = floor((x + w - k + p) / s).
__device__ __forceinline__ void erode_axis(int x, int w, int k, int s, int p, int& xo, int& wo)
{
    int first = ceil_div(x + p, s), last = floor_div(x + w - k + p, s);
    xo = first; wo = last - first + 1;
}
// Area resize n_in -> n_out: output o averages [floor(o n_in / n_out), ceil((o + 1) n_in / n_out) - 1].
__device__ __forceinline__ void resize_axis(int x, int w, int n_in, int n_out, int& xo, int& wo)
{
    int first = (int)(((long long)x * n_out + n_in - 1) / n_in);
    int last = (int)(((long long)(x + w) * n_out) / n_in) - 1;
    xo = first; wo = last - first + 1;
}

__device__ __forceinline__ dc_region empty_region() { dc_region e = {0, 0, 0, 0, 0, 0}; return e; }

__device__ dc_region apply_layer(const dc_layer_desc& L, int in_h, int in_w, dc_region a, dc_region b)
{
    if (a.w <= 0 || a.h <= 0) return empty_region();
    switch (L.kind) {
    case DC_CONV: case DC_MAXPOOL: case DC_RESIZE_AREA: {
        // D_t on the current rectangle and, independently, on the cached one; smaller size wins
        int dx, dw, dy, dh, qx, qw, qy, qh;
        if (L.kind == DC_RESIZE_AREA) {
            resize_axis(a.x, a.w, in_w, L.out_w, dx, dw);  resize_axis(a.y, a.h, in_h, L.out_h, dy, dh);
            resize_axis(a.sx, a.w, in_w, L.out_w, qx, qw); resize_axis(a.sy, a.h, in_h, L.out_h, qy, qh);
        } else {
            erode_axis(a.x, a.w, L.kw, L.sw, L.pw, dx, dw);  erode_axis(a.y, a.h, L.kh, L.sh, L.ph, dy, dh);
            erode_axis(a.sx, a.w, L.kw, L.sw, L.pw, qx, qw); erode_axis(a.sy, a.h, L.kh, L.sh, L.ph, qy, qh);
        }
        int w = min(dw, qw), h = min(dh, qh);
        if (w <= 0 || h <= 0) return empty_region();
        dc_region o = {dx, dy, w, h, qx, qy};
        return o;
    }
    case DC_LRN: {
        int r = L.ph;
        if (a.w - 2 * r <= 0 || a.h - 2 * r <= 0) return empty_region();
        dc_region o = {a.x + r, a.y + r, a.w - 2 * r, a.h - 2 * r, a.sx + r, a.sy + r};
        return o;
    }
    case DC_ADD: case DC_CONCAT: {
        // the overlapped region; both inputs must agree on the displacement
        if (b.w <= 0 || b.h <= 0) return empty_region();
        if (a.sx - a.x != b.sx - b.x || a.sy - a.y != b.sy - b.y) return empty_region();
        int x0 = max(a.x, b.x), y0 = max(a.y, b.y);
        int x1 = min(a.x + a.w, b.x + b.w), y1 = min(a.y + a.h, b.y + b.h);
        if (x1 <= x0 || y1 <= y0) return empty_region();
        dc_region o = {x0, y0, x1 - x0, y1 - y0, x0 + (a.sx - a.x), y0 + (a.sy - a.y)};
        return o;
    }
    case DC_FC:
        return empty_region();
    default:
        return a;
    }
}

__global__ void k_propagate(const dc_layer_desc* layers, const int32_t* in_hw, int layer_end, int S, int max_regions,
                            const dc_region* in, const int32_t* n_in, dc_region* table, int32_t* alive)
{
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    int s = blockIdx.y;
    if (i >= n_in[s]) return;
    const size_t slot = (size_t)s * max_regions + i;
    const size_t layer_stride = (size_t)S * max_regions;
    const dc_region r0 = in[slot];
    for (int l = 0; l < layer_end; ++l) {
        const dc_layer_desc L = layers[l];
        dc_region a = L.in0 < 0 ? r0 : table[L.in0 * layer_stride + slot];
        dc_region b = a;
        if (L.kind == DC_ADD || L.kind == DC_CONCAT) b = L.in1 < 0 ? r0 : table[L.in1 * layer_stride + slot];
        const dc_region o = apply_layer(L, in_hw[2 * l], in_hw[2 * l + 1], a, b);
        table[l * layer_stride + slot] = o;
        if (o.w > 0 && alive) atomicAdd(&alive[l * S + s], 1);     // rectangles still alive at this layer
    }
}

struct ClassifyArgs {
    const dc_region* regions; const int32_t* n_regions; int max_regions;
    const uint8_t* prev; uint8_t* out;           // maps as bytes
    int Ho, Wo, px_bytes;                        // px_bytes = cout * element size (multiple of 16)
    int tiles_x, tiles_y, S;
    uint32_t* masks; int32_t* dirty_list; int32_t* dirty_count; int32_t* reuse_px;
    const int32_t* alive;                        // per stream: rectangles alive at this layer, or NULL (unknown)
    unsigned long long* reused_total;
};

__device__ __forceinline__ void classify_tile(const ClassifyArgs& a, const int tile, const int lane)
{
    const int per = a.tiles_x * a.tiles_y;
    const int s = tile / per, t = tile - s * per, ty = t / a.tiles_x, tx = t - ty * a.tiles_x;
    const int X0 = tx * DC_TILE_W, Y0 = ty * DC_TILE_H;
    const int X1 = min(X0 + DC_TILE_W, a.Wo), Y1 = min(Y0 + DC_TILE_H, a.Ho);
    const dc_region* regs = a.regions + (size_t)s * a.max_regions;
    // every rectangle of this stream has eroded away before this layer: nothing to test or copy
    const int n = (a.alive && a.alive[s] == 0) ? 0 : a.n_regions[s];
    const size_t map_base = (size_t)s * a.Ho * a.Wo * a.px_bytes;
    uint32_t m0 = 0, m1 = 0, m2 = 0, m3 = 0;      // bit (row * DC_TILE_W + col) of the tile, row-major
    for (int base = 0; base < n; base += 32) {
        int i = base + lane;
        dc_region r = empty_region();
        int ix0 = 0, ix1 = 0, iy0 = 0, iy1 = 0;
        if (i < n) {
            r = regs[i];
            ix0 = max(r.x, X0); ix1 = min(r.x + r.w, X1);
            iy0 = max(r.y, Y0); iy1 = min(r.y + r.h, Y1);
        }
        bool hit = ix1 > ix0 && iy1 > iy0;
        if (hit) {
            const uint32_t rowbits = ((1u << (ix1 - X0)) - 1u) & ~((1u << (ix0 - X0)) - 1u);   // DC_TILE_W-bit row pattern
            for (int y = iy0; y < iy1; ++y) {
                const int bit = DC_TILE_BIT(y - Y0, 0);
                const uint32_t v = rowbits << (bit & 31);
                switch (bit >> 5) { case 0: m0 |= v; break; case 1: m1 |= v; break; case 2: m2 |= v; break; default: m3 |= v; }
            }
        }
        // the warp copies every hit span together: rows of (ix1 - ix0) pixels, px_bytes each
        unsigned hits = __ballot_sync(0xffffffffu, hit);
        while (hits) {
            int src_lane = __ffs(hits) - 1; hits &= hits - 1;
            int rx = __shfl_sync(0xffffffffu, r.x, src_lane), ry = __shfl_sync(0xffffffffu, r.y, src_lane);
            int rsx = __shfl_sync(0xffffffffu, r.sx, src_lane), rsy = __shfl_sync(0xffffffffu, r.sy, src_lane);
            int cx0 = __shfl_sync(0xffffffffu, ix0, src_lane), cx1 = __shfl_sync(0xffffffffu, ix1, src_lane);
            int cy0 = __shfl_sync(0xffffffffu, iy0, src_lane), cy1 = __shfl_sync(0xffffffffu, iy1, src_lane);
            int span_vec = (cx1 - cx0) * (a.px_bytes >> 4);          // 16-byte vectors per row
            for (int y = cy0; y < cy1; ++y) {
                const uint4* src = (const uint4*)(a.prev + map_base +
                    ((size_t)(y - ry + rsy) * a.Wo + (cx0 - rx + rsx)) * a.px_bytes);
                uint4* dst = (uint4*)(a.out + map_base + ((size_t)y * a.Wo + cx0) * a.px_bytes);
                for (int v = lane; v < span_vec; v += 32) dst[v] = __ldg(src + v);
            }
        }
    }
    m0 = __reduce_or_sync(0xffffffffu, m0); m1 = __reduce_or_sync(0xffffffffu, m1);
    m2 = __reduce_or_sync(0xffffffffu, m2); m3 = __reduce_or_sync(0xffffffffu, m3);
    if (lane == 0) {
        uint32_t* mk = a.masks + (size_t)tile * 4;
        mk[0] = m0; mk[1] = m1; mk[2] = m2; mk[3] = m3;
        int covered = __popc(m0) + __popc(m1) + __popc(m2) + __popc(m3);
        int in_tile = (X1 - X0) * (Y1 - Y0);
        if (covered) { atomicAdd(&a.reuse_px[s], covered); atomicAdd(a.reused_total, (unsigned long long)covered); }
        if (covered < in_tile) {
            int slot = atomicAdd(a.dirty_count, 1);
            a.dirty_list[slot] = tile;
        }
    }
}

__global__ void __launch_bounds__(256) k_classify_copy(ClassifyArgs a)
{
    const int tile = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (tile >= a.tiles_x * a.tiles_y * a.S) return;
    classify_tile(a, tile, threadIdx.x & 31);
}

// Every cached layer of a frame in one launch: the bitmaps, reuse copies and dirty lists of a layer depend only
// on the rectangles (known once propagation has run) and on the layer's own cached map, not on the layers before it.
// Warps are numbered through all layers' tiles; first_warp is the running sum.
struct ClassifyLayer {
    const dc_region* regions; uint8_t* map[2];
    int Ho, Wo, px_bytes, tiles_x, tiles_y, first_warp;
    uint32_t* masks; int32_t* dirty_list; int32_t* dirty_count; int32_t* reuse_px;
    const int32_t* alive; unsigned long long* reused_total;
};

__global__ void __launch_bounds__(256) k_classify_copy_all(const ClassifyLayer* layers, int n_cached, int total_warps,
                                                           const int32_t* n_regions, int max_regions, int S, int cur)
{
    const int w = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (w >= total_warps) return;
    int lo = 0, hi = n_cached - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (layers[mid].first_warp <= w) lo = mid; else hi = mid - 1;
    }
    const ClassifyLayer& L = layers[lo];
    ClassifyArgs a;
    a.regions = L.regions; a.n_regions = n_regions; a.max_regions = max_regions;
    a.prev = L.map[cur]; a.out = L.map[cur ^ 1];
    a.Ho = L.Ho; a.Wo = L.Wo; a.px_bytes = L.px_bytes; a.tiles_x = L.tiles_x; a.tiles_y = L.tiles_y; a.S = S;
    a.masks = L.masks; a.dirty_list = L.dirty_list; a.dirty_count = L.dirty_count; a.reuse_px = L.reuse_px;
    a.alive = L.alive; a.reused_total = L.reused_total;
    classify_tile(a, w - L.first_warp, threadIdx.x & 31);
}

}  // namespace

// Builds the device table for k_classify_copy_all (once, after every map is allocated).
int dc_build_classify_table(dc_cache* c)
{
    const int n = c->n_layers;
    ClassifyLayer* h = (ClassifyLayer*)malloc(sizeof(ClassifyLayer) * (n > 0 ? n : 1));
    if (!h) return DC_ERR_ALLOC;
    int k = 0, warps = 0;
    for (int i = 0; i < n; ++i) {
        if (!dc_layer_cached(c, i)) continue;
        dc_layer_rt& L = c->L[i];
        ClassifyLayer& e = h[k++];
        e.regions = c->table + (size_t)i * c->S * c->max_regions;
        e.map[0] = (uint8_t*)L.map[0]; e.map[1] = (uint8_t*)L.map[1];
        e.Ho = L.d.out_h; e.Wo = L.d.out_w; e.px_bytes = L.d.cout * c->elt;
        e.tiles_x = L.tiles_x; e.tiles_y = L.tiles_y; e.first_warp = warps;
        e.masks = L.masks; e.dirty_list = L.dirty_list; e.dirty_count = c->dirty_count + i;
        e.reuse_px = c->reuse_px + (size_t)i * c->S; e.alive = c->alive + (size_t)i * c->S;
        e.reused_total = c->reused_total + i;
        warps += L.tiles_x * L.tiles_y * c->S;
    }
    c->n_cached = k; c->classify_warps = warps;
    int rc = DC_OK;
    if (k > 0) {
        if (cudaMalloc(&c->classify_table, sizeof(ClassifyLayer) * k) != cudaSuccess) { cudaGetLastError(); rc = DC_ERR_ALLOC; }
        else if (cudaMemcpy(c->classify_table, h, sizeof(ClassifyLayer) * k, cudaMemcpyHostToDevice) != cudaSuccess) rc = DC_ERR_CUDA;
        else c->bytes += sizeof(ClassifyLayer) * k;
    }
    free(h);
    return rc;
}

// All cached layers at once; `cur` is the index of the map that holds the cached values (the same for every layer:
// they all flip once per frame).  The caller has zeroed the dirty counts and the reuse counters on the stream.
int dc_launch_classify_all(dc_cache* c, int cur)
{
    if (c->n_cached <= 0) return DC_OK;
    {
        dc_prof_scope ps(c, DC_ST_CLASSIFY_COPY);
        k_classify_copy_all<<<dc_div_up(c->classify_warps, 8), 256, 0, c->stream>>>(
            (const ClassifyLayer*)c->classify_table, c->n_cached, c->classify_warps, c->n_regions, c->max_regions, c->S, cur);
    }
    c->launches += 1;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}

int dc_launch_propagate(dc_cache* c, const dc_region* in, const int32_t* n_in, int layer_end)
{
    dim3 grid(dc_div_up(c->max_regions, 128), c->S);
    {
        dc_prof_scope ps(c, DC_ST_PROPAGATE);
        k_propagate<<<grid, 128, 0, c->stream>>>(c->layers_dev, c->in_hw_dev, layer_end, c->S, c->max_regions,
                                                 in, n_in, c->table, c->alive);
    }
    c->launches += 1;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}

int dc_launch_classify_copy(dc_cache* c, int layer, const dc_region* regions, const int32_t* n_regions,
                            const void* prev_out, void* out)
{
    dc_layer_rt& L = c->L[layer];
    ClassifyArgs a;
    a.regions = regions; a.n_regions = n_regions; a.max_regions = c->max_regions;
    a.prev = (const uint8_t*)prev_out; a.out = (uint8_t*)out;
    a.Ho = L.d.out_h; a.Wo = L.d.out_w; a.px_bytes = L.d.cout * c->elt;
    a.tiles_x = L.tiles_x; a.tiles_y = L.tiles_y; a.S = c->S;
    a.masks = L.masks; a.dirty_list = L.dirty_list; a.dirty_count = c->dirty_count + layer;
    a.reuse_px = c->reuse_px + (size_t)layer * c->S;
    a.reused_total = c->reused_total + layer;
    a.alive = (regions == c->table + (size_t)layer * c->S * c->max_regions) ? c->alive + (size_t)layer * c->S : nullptr;
    // the caller has zeroed dirty_count[layer] and reuse_px[layer][*] on the stream
    int tiles = L.tiles_x * L.tiles_y * c->S;
    { dc_prof_scope ps(c, DC_ST_CLASSIFY_COPY); k_classify_copy<<<dc_div_up(tiles, 8), 256, 0, c->stream>>>(a); }
    c->launches += 1;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}
