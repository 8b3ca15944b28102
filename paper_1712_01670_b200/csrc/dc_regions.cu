// Region propagation (Section 5, Table 2) and the reuse step of the cache-aware convolution
// (Section 5, "Reuse": copy cached regions, build the bitmap, list what is left to compute).
//
//   k_propagate      one thread per (stream, rectangle slot) walks the layer table in order and
//                    writes the rectangle's image after every layer.  Slots are independent,
//                    so no synchronisation is needed; a vanished rectangle is all zeros.
//   k_classify_copy  one warp per 16x8 output tile: lanes test the stream's rectangles against
//                    the tile, OR their coverage into a 128-bit bitmap, the warp copies each
//                    covered row span from the cached map with bulk copies (global -> shared ->
//                    global through the copy engine, no registers), and tiles that still hold
//                    uncovered pixels are appended to the layer's dirty list.
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
    if (i >= max_regions || i >= n_in[s]) return;          // a caller's count beyond the table is cut, never written
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

// ---- bulk copies (cp.async.bulk) for the reuse copy ----
#ifndef DC_COPY_WARPS
#define DC_COPY_WARPS 8
#endif
#ifndef DC_COPY_SEG
#define DC_COPY_SEG 256
#endif
constexpr int kCopyWarps = DC_COPY_WARPS;        // warps per CTA
constexpr int kSeg = DC_COPY_SEG;                // bytes one lane moves per round; a row span is cut into such segments
constexpr int kStageBytes = 32 * kSeg;           // staging of one warp: one segment per lane
constexpr size_t kCopySmem = (size_t)kCopyWarps * kStageBytes + 128 + kCopyWarps * sizeof(unsigned long long);
constexpr unsigned long long kCopyWaitNs = 2000000000ull;   // a warp gives up on its staging barrier after 2 s (far beyond any copy)

__device__ __forceinline__ uint32_t rs_smem(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void rs_bar_init(void* bar)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(rs_smem(bar)) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void rs_expect(void* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(rs_smem(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool rs_try(void* bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(rs_smem(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ void rs_load(void* dst_smem, const void* src, uint32_t bytes, void* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(rs_smem(dst_smem)), "l"(src), "r"(bytes), "r"(rs_smem(bar)) : "memory");
}
__device__ __forceinline__ void rs_store(void* dst, const void* src_smem, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(rs_smem(src_smem)), "r"(bytes) : "memory");
}
__device__ __forceinline__ unsigned long long rs_now()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait for a phase of the staging barrier; false when the limit passed.
__device__ __forceinline__ bool rs_wait(void* bar, uint32_t parity)
{
    if (rs_try(bar, parity)) return true;
    const unsigned long long t0 = rs_now();
    for (unsigned spin = 1;; ++spin) {
        if (rs_try(bar, parity)) return true;
        if ((spin & 255u) == 0 && rs_now() - t0 > kCopyWaitNs) return false;
    }
}
__device__ __forceinline__ void rs_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void rs_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void rs_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// What a warp needs for its bulk copies: its staging (32 segments), one mbarrier and its phase.
struct CopyLane { uint8_t* stage; unsigned long long* bar; uint32_t phase; bool dead; };

struct ClassifyArgs {
    const dc_region* regions; const int32_t* n_regions; int max_regions;
    const uint8_t* prev; uint8_t* out;           // maps as bytes
    int Ho, Wo, px_bytes;                        // px_bytes = cout * element size (multiple of 16)
    int tiles_x, tiles_y, S;
    int gpr, n_tiles;                            // gpr > 0: flat tiles of 16 groups of 8 pixels, gpr groups per image row; n_tiles: tiles in all
    uint32_t* masks; int32_t* dirty_list; int32_t* dirty_count; int32_t* reuse_px;
    const int32_t* alive;                        // per stream: rectangles alive at this layer, or NULL (unknown)
    unsigned long long* reused_total;
    int32_t* status;                             // device status word
};

__device__ __forceinline__ void classify_tile(const ClassifyArgs& a, const int tile, const int lane, CopyLane& cl)
{
    const int per = a.tiles_x * a.tiles_y;
    const int s = tile / per, t = tile - s * per, ty = t / a.tiles_x, tx = t - ty * a.tiles_x;
    const int X0 = tx * DC_TILE_W, Y0 = ty * DC_TILE_H;
    const int X1 = min(X0 + DC_TILE_W, a.Wo), Y1 = min(Y0 + DC_TILE_H, a.Ho);
    const dc_region* regs = a.regions + (size_t)s * a.max_regions;
    // every rectangle of this stream has eroded away before this layer: nothing to test or copy
    const int n = (a.alive && a.alive[s] == 0) ? 0 : min(a.n_regions[s], a.max_regions);
    const size_t map_base = (size_t)s * a.Ho * a.Wo * a.px_bytes;
    uint32_t m0 = 0, m1 = 0, m2 = 0, m3 = 0;      // bit (row * DC_TILE_W + col) of the tile, row-major
    for (int base = 0; base < n; base += 32) {
        int i = base + lane;
        dc_region r = empty_region();
        int ix0 = 0, ix1 = 0, iy0 = 0, iy1 = 0;
        if (i < n) {
            r = regs[i];
            // Rectangles made by Step 5 and Table 2 lie inside the map on both sides.  One that does not (a caller's
            // own list) is not reused: neither side is ever addressed outside its map; the status word records it.
            const bool inside = r.x >= 0 && r.y >= 0 && r.sx >= 0 && r.sy >= 0 && r.w <= a.Wo && r.h <= a.Ho &&
                                r.x <= a.Wo - r.w && r.y <= a.Ho - r.h && r.sx <= a.Wo - r.w && r.sy <= a.Ho - r.h;
            if (r.w <= 0 || r.h <= 0) r = empty_region();
            else if (!inside) {
                if (t == 0 && a.status) atomicExch(a.status, (int)DC_ERR_ARG);
                r = empty_region();
            }
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
            // Section 5 "Reuse", step 1.  Inside the tile the rectangle is (cy1 - cy0) row spans, each contiguous in both
            // maps (all channels of cx1 - cx0 pixels).  Spans are cut into segments of kSeg bytes; per round every lane
            // moves one segment: a bulk copy into the warp's staging, then a bulk copy out to the new map.  Addresses
            // and sizes are multiples of 16 bytes (px_bytes is).
            const int span_bytes = (cx1 - cx0) * a.px_bytes;
            const int segs = (span_bytes + kSeg - 1) / kSeg, items = (cy1 - cy0) * segs;
            const uint8_t* src0 = a.prev + map_base + ((size_t)(cy0 - ry + rsy) * a.Wo + (cx0 - rx + rsx)) * a.px_bytes;
            uint8_t* dst0 = a.out + map_base + ((size_t)cy0 * a.Wo + cx0) * a.px_bytes;
            const size_t row_pitch = (size_t)a.Wo * a.px_bytes;
            for (int i0 = 0; i0 < items && !cl.dead; i0 += 32) {
                const int it = i0 + lane;
                const bool on = it < items;
                const int row = on ? it / segs : 0, sg = it - row * segs;
                const uint32_t bytes = on ? (uint32_t)min(kSeg, span_bytes - sg * kSeg) : 0u;
                const size_t off = (size_t)row * row_pitch + (size_t)sg * kSeg;
                const uint32_t total = __reduce_add_sync(0xffffffffu, bytes);
                if (lane == 0) rs_expect(cl.bar, total);
                __syncwarp();
                if (on) rs_load(cl.stage + lane * kSeg, src0 + off, bytes, cl.bar);
                const bool landed = rs_wait(cl.bar, cl.phase);
                if (!__all_sync(0xffffffffu, landed)) {                     // never seen; leave rather than spin for ever
                    if (lane == 0 && a.status) atomicExch(a.status, (int)DC_ERR_TIMEOUT);
                    cl.dead = true;
                    break;
                }
                cl.phase ^= 1u;
                if (on) rs_store(dst0 + off, cl.stage + lane * kSeg, bytes);
                rs_commit();
                rs_wait_read();                                             // staging may be overwritten by the next round
                __syncwarp();
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


// The same for a layer with flat tiles: row i of the tile's bitmap is group tile * 16 + i, a group being 8 pixels of
// one image row, numbered (stream * Ho + y) * gpr + column group.  A tile may hold groups of several streams (small
// maps); each stream's rectangles are tested against that stream's groups only.
__device__ __forceinline__ void classify_tile_flat(const ClassifyArgs& a, const int tile, const int lane, CopyLane& cl)
{
    const int gps = a.Ho * a.gpr;                                  // groups per stream
    const int G0 = tile * DC_TILE_H, G1 = min(G0 + DC_TILE_H, a.S * gps);
    uint32_t m0 = 0, m1 = 0, m2 = 0, m3 = 0;
    int in_tile;
    {   // pixels of the tile that exist: a row's last group may be cut by the map's width
        const int g = G0 + lane, loc = g % gps, gx = loc % a.gpr;
        in_tile = __reduce_add_sync(0xffffffffu, (lane < DC_TILE_H && g < G1) ? min(DC_TILE_W, a.Wo - gx * DC_TILE_W) : 0);
    }
    const int segs_max = (DC_TILE_W * a.px_bytes + kSeg - 1) / kSeg;   // segments of a whole group's pixels
    for (int s = G0 / gps; s * gps < G1; ++s) {
        const int g_lo = max(G0, s * gps), g_hi = min(G1, (s + 1) * gps);     // this stream's groups in the tile
        const int loc0 = g_lo - s * gps, y_first = loc0 / a.gpr, gx_first = loc0 - y_first * a.gpr;
        const dc_region* regs = a.regions + (size_t)s * a.max_regions;
        const int n = (a.alive && a.alive[s] == 0) ? 0 : min(a.n_regions[s], a.max_regions);
        const size_t map_base = (size_t)s * a.Ho * a.Wo * a.px_bytes;
        uint32_t s0 = 0, s1 = 0, s2 = 0, s3 = 0;                  // this stream's part of the bitmap
        for (int base = 0; base < n; base += 32) {
            const int i = base + lane;
            dc_region r = empty_region();
            uint32_t hit16 = 0;                                   // rows of the tile that the rectangle touches
            if (i < n) {
                r = regs[i];
                const bool inside = r.x >= 0 && r.y >= 0 && r.sx >= 0 && r.sy >= 0 && r.w <= a.Wo && r.h <= a.Ho &&
                                    r.x <= a.Wo - r.w && r.y <= a.Ho - r.h && r.sx <= a.Wo - r.w && r.sy <= a.Ho - r.h;
                if (r.w <= 0 || r.h <= 0) r = empty_region();
                else if (!inside) {                               // see classify_tile
                    if (loc0 == 0 && a.status) atomicExch(a.status, (int)DC_ERR_ARG);
                    r = empty_region();
                }
                if (r.w > 0) {
                    int y = y_first, gx = gx_first;
                    for (int g = g_lo; g < g_hi; ++g) {
                        const int x0 = gx * DC_TILE_W;
                        const int cx0 = max(r.x, x0), cx1 = min(r.x + r.w, min(x0 + DC_TILE_W, a.Wo));
                        if (y >= r.y && y < r.y + r.h && cx1 > cx0) {
                            const int row = g - G0;
                            const uint32_t v = (((1u << (cx1 - x0)) - 1u) & ~((1u << (cx0 - x0)) - 1u)) << ((row & 3) * DC_TILE_W);
                            switch (row >> 2) { case 0: s0 |= v; break; case 1: s1 |= v; break; case 2: s2 |= v; break; default: s3 |= v; }
                            hit16 |= 1u << row;
                        }
                        if (++gx == a.gpr) { gx = 0; ++y; }
                    }
                }
            }
            // the warp copies every touched row's span together (Section 5 "Reuse", step 1): per round one segment per lane
            unsigned hits = __ballot_sync(0xffffffffu, hit16 != 0);
            while (hits) {
                const int src_lane = __ffs(hits) - 1; hits &= hits - 1;
                const int rx = __shfl_sync(0xffffffffu, r.x, src_lane), ry = __shfl_sync(0xffffffffu, r.y, src_lane);
                const int rw = __shfl_sync(0xffffffffu, r.w, src_lane);
                const int rsx = __shfl_sync(0xffffffffu, r.sx, src_lane), rsy = __shfl_sync(0xffffffffu, r.sy, src_lane);
                const uint32_t h16 = __shfl_sync(0xffffffffu, hit16, src_lane);
                for (int i0 = 0; i0 < DC_TILE_H * segs_max && !cl.dead; i0 += 32) {
                    const int it = i0 + lane, row = it / segs_max, sg = it - row * segs_max;
                    uint32_t bytes = 0;
                    size_t src_off = 0, dst_off = 0;
                    if (row < DC_TILE_H && ((h16 >> row) & 1u)) {
                        const int loc = G0 + row - s * gps, y = loc / a.gpr, x0 = (loc - y * a.gpr) * DC_TILE_W;
                        const int cx0 = max(rx, x0), cx1 = min(rx + rw, min(x0 + DC_TILE_W, a.Wo));
                        const int span = (cx1 - cx0) * a.px_bytes - sg * kSeg;
                        if (span > 0) {
                            bytes = (uint32_t)min(kSeg, span);
                            src_off = ((size_t)(y - ry + rsy) * a.Wo + (cx0 - rx + rsx)) * a.px_bytes + (size_t)sg * kSeg;
                            dst_off = ((size_t)y * a.Wo + cx0) * a.px_bytes + (size_t)sg * kSeg;
                        }
                    }
                    const uint32_t total = __reduce_add_sync(0xffffffffu, bytes);
                    if (total == 0) continue;                     // the same in all lanes
                    if (lane == 0) rs_expect(cl.bar, total);
                    __syncwarp();
                    if (bytes) rs_load(cl.stage + lane * kSeg, a.prev + map_base + src_off, bytes, cl.bar);
                    const bool landed = rs_wait(cl.bar, cl.phase);
                    if (!__all_sync(0xffffffffu, landed)) {
                        if (lane == 0 && a.status) atomicExch(a.status, (int)DC_ERR_TIMEOUT);
                        cl.dead = true;
                        break;
                    }
                    cl.phase ^= 1u;
                    if (bytes) rs_store(a.out + map_base + dst_off, cl.stage + lane * kSeg, bytes);
                    rs_commit();
                    rs_wait_read();
                    __syncwarp();
                }
            }
        }
        s0 = __reduce_or_sync(0xffffffffu, s0); s1 = __reduce_or_sync(0xffffffffu, s1);
        s2 = __reduce_or_sync(0xffffffffu, s2); s3 = __reduce_or_sync(0xffffffffu, s3);
        const int covered_s = __popc(s0) + __popc(s1) + __popc(s2) + __popc(s3);
        if (lane == 0 && covered_s) { atomicAdd(&a.reuse_px[s], covered_s); atomicAdd(a.reused_total, (unsigned long long)covered_s); }
        m0 |= s0; m1 |= s1; m2 |= s2; m3 |= s3;
    }
    if (lane == 0) {
        uint32_t* mk = a.masks + (size_t)tile * 4;
        mk[0] = m0; mk[1] = m1; mk[2] = m2; mk[3] = m3;
        if (__popc(m0) + __popc(m1) + __popc(m2) + __popc(m3) < in_tile) {
            const int slot = atomicAdd(a.dirty_count, 1);
            a.dirty_list[slot] = tile;
        }
    }
}

// Staging and barrier of this warp, carved from the CTA's dynamic shared memory.
__device__ __forceinline__ CopyLane copy_lane_setup(uint8_t* smem_raw)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t* base = (uint8_t*)(((uintptr_t)smem_raw + 127) & ~(uintptr_t)127);
    CopyLane cl;
    cl.stage = base + (size_t)warp * kStageBytes;
    cl.bar = (unsigned long long*)(base + (size_t)kCopyWarps * kStageBytes) + warp;
    cl.phase = 0; cl.dead = false;
    if (lane == 0) rs_bar_init(cl.bar);
    __syncwarp();
    return cl;
}

__global__ void __launch_bounds__(kCopyWarps * 32) k_classify_copy(ClassifyArgs a)
{
    extern __shared__ uint8_t copy_smem[];
    CopyLane cl = copy_lane_setup(copy_smem);
    const int tile = blockIdx.x * kCopyWarps + (threadIdx.x >> 5);
    if (tile < a.n_tiles) {
        if (a.gpr > 0) classify_tile_flat(a, tile, threadIdx.x & 31, cl);
        else classify_tile(a, tile, threadIdx.x & 31, cl);
    }
    rs_wait_all();
}

// Every cached layer of a frame in one launch: the bitmaps, reuse copies and dirty lists of a layer depend only
// on the rectangles (known once propagation has run) and on the layer's own cached map, not on the layers before it.
// Warps are numbered through all layers' tiles; first_warp is the running sum.
struct ClassifyLayer {
    const dc_region* regions; uint8_t* map[2];
    int Ho, Wo, px_bytes, tiles_x, tiles_y, first_warp, gpr;
    uint32_t* masks; int32_t* dirty_list; int32_t* dirty_count; int32_t* reuse_px;
    const int32_t* alive; unsigned long long* reused_total; int32_t* status;
};

__global__ void __launch_bounds__(kCopyWarps * 32) k_classify_copy_all(const ClassifyLayer* layers, int n_cached, int total_warps,
                                                                       const int32_t* n_regions, int max_regions, int S, int cur)
{
    extern __shared__ uint8_t copy_smem[];
    CopyLane cl = copy_lane_setup(copy_smem);
    const int w = blockIdx.x * kCopyWarps + (threadIdx.x >> 5);
    if (w >= total_warps) return;                       // no copy was issued by this warp
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
    a.gpr = L.gpr; a.n_tiles = 0;
    a.masks = L.masks; a.dirty_list = L.dirty_list; a.dirty_count = L.dirty_count; a.reuse_px = L.reuse_px;
    a.alive = L.alive; a.reused_total = L.reused_total; a.status = L.status;
    if (a.gpr > 0) classify_tile_flat(a, w - L.first_warp, threadIdx.x & 31, cl);
    else classify_tile(a, w - L.first_warp, threadIdx.x & 31, cl);
    rs_wait_all();
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
        e.gpr = L.flat ? L.gpr : 0;
        e.masks = L.masks; e.dirty_list = L.dirty_list; e.dirty_count = c->dirty_count + i;
        e.reuse_px = c->reuse_px + (size_t)i * c->S; e.alive = c->alive + (size_t)i * c->S;
        e.reused_total = c->reused_total + i;
        e.status = c->status;
        warps += dc_layer_tiles(c, L);
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
        static dc_once_per_device attr_set;
        if (attr_set.first(c->device))
            DC_CUDA(cudaFuncSetAttribute(k_classify_copy_all, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kCopySmem));
        k_classify_copy_all<<<dc_div_up(c->classify_warps, kCopyWarps), kCopyWarps * 32, kCopySmem, c->stream>>>(
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
    a.gpr = L.flat ? L.gpr : 0; a.n_tiles = dc_layer_tiles(c, L);
    a.masks = L.masks; a.dirty_list = L.dirty_list; a.dirty_count = c->dirty_count + layer;
    a.reuse_px = c->reuse_px + (size_t)layer * c->S;
    a.reused_total = c->reused_total + layer;
    a.status = c->status;
    a.alive = (regions == c->table + (size_t)layer * c->S * c->max_regions) ? c->alive + (size_t)layer * c->S : nullptr;
    // the caller has zeroed dirty_count[layer] and reuse_px[layer][*] on the stream
    int tiles = dc_layer_tiles(c, L);
    static dc_once_per_device attr_set;
    if (attr_set.first(c->device))
        DC_CUDA(cudaFuncSetAttribute(k_classify_copy, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kCopySmem));
    { dc_prof_scope ps(c, DC_ST_CLASSIFY_COPY); k_classify_copy<<<dc_div_up(tiles, kCopyWarps), kCopyWarps * 32, kCopySmem, c->stream>>>(a); }
    c->launches += 1;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}
