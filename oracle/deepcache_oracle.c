/*
 * CPU oracle for the DeepCache per-frame hot path (arXiv 1712.01670).
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow, obviously-correct C that restates
 * the paper's steps one by one.  It shares no code with the CUDA library and
 * must never be called from the product path; only the tests, the smoke check
 * and the benchmark's CPU-baseline leg may use it.
 *
 * Conventions
 *   frames   uint8, HWC (3 channels), row pitch in bytes
 *   maps     double, NHWC (one stream at a time: HWC)
 *   weights  double, [cout][kh][kw][cin] ([cout][kh][kw][cin / groups] for a grouped convolution)
 *   motion   MV = (dx, dy) points from a block of the current frame to its
 *            match in the previous frame: previous = current + MV
 *            (Section 4, Step 2: (x'_i - x_i, y'_i - y_i))
 *   region   destination rectangle (x, y, w, h) in the current map and the
 *            origin (sx, sy) of the same-sized source rectangle in the cached
 *            map (Section 3, "(x, y, w, h) -> (x', y', w, h)")
 *
 * OpenMP pragmas only spread independent outer loops over cores for timing;
 * they change no result.
 *
 * Pins (tests/test_oracle_*.py): brute-force search on tiny frames, the PSNR
 * closed form at T = 20, the Fig. 7 and Section 4 erosion examples, composed
 * receptive-field closed form, boolean dependency tracing, torch conv2d /
 * max_pool2d / adaptive_avg_pool2d in float64, identical-frame and all-dirty
 * special cases.  The diamond-search walk itself has no printed example in
 * the paper: beyond its invariants it is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct { int32_t x, y, w, h, sx, sy; } orc_region;

typedef struct {
    int32_t kind, kh, kw, sh, sw, ph, pw, cin, cout, relu, in0, in1, out_h, out_w;
    int32_t groups;   /* convolution only: the channels are cut into this many independent groups (0 or 1: one) */
} orc_layer;

enum { ORC_CONV = 0, ORC_MAXPOOL = 1, ORC_RELU = 2, ORC_ADD = 3, ORC_CONCAT = 4,
       ORC_RESIZE_AREA = 5, ORC_LRN = 6, ORC_FC = 7 };

#define ORC_INVALID UINT64_MAX

/* ------------------------------------------------------------------------
 * Section 4, Step 2: block similarity
 * ---------------------------------------------------------------------- */

/* Sum of squared differences between the current-frame block at (x0, y0),
 * size bw x bh, and the previous-frame block displaced by (dx, dy), over all
 * three channels.  A displaced block that leaves the frame is not a candidate. */
uint64_t orc_block_sse(const uint8_t* cur, const uint8_t* prev, int W, int H, int64_t pitch,
                       int x0, int y0, int bw, int bh, int dx, int dy)
{
    if (x0 + dx < 0 || y0 + dy < 0 || x0 + dx + bw > W || y0 + dy + bh > H) return ORC_INVALID;
    uint64_t sse = 0;
    for (int y = 0; y < bh; ++y)
        for (int x = 0; x < bw; ++x)
            for (int c = 0; c < 3; ++c) {
                int a = cur[(int64_t)(y0 + y) * pitch + (x0 + x) * 3 + c];
                int b = prev[(int64_t)(y0 + dy + y) * pitch + (x0 + dx + x) * 3 + c];
                sse += (uint64_t)((a - b) * (a - b));
            }
    return sse;
}

/* PSNR = 10 log10(255^2 / MSE), MSE = SSE / n (Step 2).  PSNR > T  <=>
 * SSE < 65025 n / 10^(T/10).  Returns the largest integer SSE that passes. */
int64_t orc_psnr_limit(int64_t n, double T)
{
    double q = 65025.0 * (double)n / pow(10.0, T / 10.0);
    return (int64_t)ceil(q) - 1;
}

int orc_psnr_pass(uint64_t sse, int64_t n, double T)
{
    if (sse == ORC_INVALID) return 0;
    return (int64_t)sse <= orc_psnr_limit(n, T);
}

/* Total order on candidates: smaller SSE first; ties go to the smaller
 * |dx| + |dy|, then the smaller dy, then the smaller dx. */
static int key_less(uint64_t sa, int dxa, int dya, uint64_t sb, int dxb, int dyb)
{
    if (sa != sb) return sa < sb;
    int la = abs(dxa) + abs(dya), lb = abs(dxb) + abs(dyb);
    if (la != lb) return la < lb;
    if (dya != dyb) return dya < dyb;
    return dxa < dxb;
}

static void block_geom(int W, int H, int B, int bx, int by, int* x0, int* y0, int* bw, int* bh)
{
    *x0 = bx * B; *y0 = by * B;
    *bw = (W - *x0 < B) ? W - *x0 : B;     /* Step 1: edge blocks are clipped */
    *bh = (H - *y0 < B) ? H - *y0 : B;
}

/* Exhaustive search: every displacement with |dx|, |dy| <= R. */
static void search_es(const uint8_t* cur, const uint8_t* prev, int W, int H, int64_t pitch,
                      int x0, int y0, int bw, int bh, int R, int* bdx, int* bdy, uint64_t* bsse)
{
    uint64_t best = ORC_INVALID; int bx = 0, by = 0;
    for (int dy = -R; dy <= R; ++dy)
        for (int dx = -R; dx <= R; ++dx) {
            uint64_t s = orc_block_sse(cur, prev, W, H, pitch, x0, y0, bw, bh, dx, dy);
            if (s == ORC_INVALID) continue;
            if (best == ORC_INVALID || key_less(s, dx, dy, best, bx, by)) { best = s; bx = dx; by = dy; }
        }
    *bdx = bx; *bdy = by; *bsse = best;
}

/* Diamond search (Zhu & Ma, cited in Step 2).  Large diamond = centre plus
 * (0,+-2), (+-2,0), (+-1,+-1); recentre on the best point until the centre is
 * best; then the small diamond (0,+-1), (+-1,0) gives the result.  Points
 * outside the frame or beyond +-R are skipped. */
static void search_ds(const uint8_t* cur, const uint8_t* prev, int W, int H, int64_t pitch,
                      int x0, int y0, int bw, int bh, int R, int* bdx, int* bdy, uint64_t* bsse)
{
    static const int large[8][2] = { {0,-2}, {-1,-1}, {1,-1}, {-2,0}, {2,0}, {-1,1}, {1,1}, {0,2} };
    static const int small[4][2] = { {0,-1}, {-1,0}, {1,0}, {0,1} };
    int cx = 0, cy = 0;
    uint64_t cs = orc_block_sse(cur, prev, W, H, pitch, x0, y0, bw, bh, 0, 0);
    for (;;) {
        int nx = cx, ny = cy; uint64_t ns = cs;
        for (int i = 0; i < 8; ++i) {
            int dx = cx + large[i][0], dy = cy + large[i][1];
            if (abs(dx) > R || abs(dy) > R) continue;
            uint64_t s = orc_block_sse(cur, prev, W, H, pitch, x0, y0, bw, bh, dx, dy);
            if (s == ORC_INVALID) continue;
            if (key_less(s, dx, dy, ns, nx, ny)) { ns = s; nx = dx; ny = dy; }
        }
        if (nx == cx && ny == cy) break;
        cx = nx; cy = ny; cs = ns;
    }
    int nx = cx, ny = cy; uint64_t ns = cs;
    for (int i = 0; i < 4; ++i) {
        int dx = cx + small[i][0], dy = cy + small[i][1];
        if (abs(dx) > R || abs(dy) > R) continue;
        uint64_t s = orc_block_sse(cur, prev, W, H, pitch, x0, y0, bw, bh, dx, dy);
        if (s == ORC_INVALID) continue;
        if (key_less(s, dx, dy, ns, nx, ny)) { ns = s; nx = dx; ny = dy; }
    }
    *bdx = nx; *bdy = ny; *bsse = ns;
}

/* Three step search (named in Section 7.5 as an alternative unit for Step 2; its definition is the
 * classic one from the block-matching literature the paper cites).  Around the current centre the
 * eight points at (+-S, 0), (0, +-S), (+-S, +-S) are scored; the best of the nine becomes the centre;
 * S halves; the pass with S = 1 gives the result.  The first step is the largest power of two S0
 * with 2 S0 - 1 <= R (R = 7 gives the textbook 4, 2, 1), so no visited point lies beyond +-R by
 * construction of the sum S0 + S0/2 + ... + 1; points outside the frame are skipped, and the bound
 * on |d| is still checked for R that are not of the form 2^n - 1. */
static void search_tss(const uint8_t* cur, const uint8_t* prev, int W, int H, int64_t pitch,
                       int x0, int y0, int bw, int bh, int R, int* bdx, int* bdy, uint64_t* bsse)
{
    int S = 1;
    while (2 * (2 * S) - 1 <= R) S *= 2;
    if (R < 1) S = 0;
    int cx = 0, cy = 0;
    uint64_t cs = orc_block_sse(cur, prev, W, H, pitch, x0, y0, bw, bh, 0, 0);
    for (; S >= 1; S /= 2) {
        int nx = cx, ny = cy; uint64_t ns = cs;
        for (int j = -1; j <= 1; ++j)
            for (int i = -1; i <= 1; ++i) {
                if (i == 0 && j == 0) continue;
                int dx = cx + i * S, dy = cy + j * S;
                if (abs(dx) > R || abs(dy) > R) continue;
                uint64_t s = orc_block_sse(cur, prev, W, H, pitch, x0, y0, bw, bh, dx, dy);
                if (s == ORC_INVALID) continue;
                if (key_less(s, dx, dy, ns, nx, ny)) { ns = s; nx = dx; ny = dy; }
            }
        cx = nx; cy = ny; cs = ns;
    }
    *bdx = cx; *bdy = cy; *bsse = cs;
}

#define ORC_NOT_SEARCHED UINT32_MAX

/* Step 2 for the blocks of the grid.  kind: 0 exhaustive, 1 diamond, 2 three step.
 * mv is [Gy][Gx][2] = (dx, dy); sse is [Gy][Gx].
 * skip_k (Section 4, the k-skip acceleration): only blocks whose row and column index are
 * multiples of skip_k are searched; the others get mv = (0, 0), sse = ORC_NOT_SEARCHED and take
 * no part in Step 3.  skip_k = 1 searches every block. */
void orc_search_k(const uint8_t* cur, const uint8_t* prev, int W, int H, int64_t pitch,
                  int B, int R, int kind, int skip_k, int16_t* mv, uint32_t* sse)
{
    int Gx = (W + B - 1) / B, Gy = (H + B - 1) / B;
    #pragma omp parallel for schedule(dynamic, 4)
    for (int b = 0; b < Gx * Gy; ++b) {
        int bx = b % Gx, by = b / Gx, x0, y0, bw, bh, dx, dy; uint64_t s;
        if (bx % skip_k != 0 || by % skip_k != 0) { mv[2 * b] = 0; mv[2 * b + 1] = 0; sse[b] = ORC_NOT_SEARCHED; continue; }
        block_geom(W, H, B, bx, by, &x0, &y0, &bw, &bh);
        if (kind == 0) search_es(cur, prev, W, H, pitch, x0, y0, bw, bh, R, &dx, &dy, &s);
        else if (kind == 2) search_tss(cur, prev, W, H, pitch, x0, y0, bw, bh, R, &dx, &dy, &s);
        else           search_ds(cur, prev, W, H, pitch, x0, y0, bw, bh, R, &dx, &dy, &s);
        mv[2 * b] = (int16_t)dx; mv[2 * b + 1] = (int16_t)dy; sse[b] = (uint32_t)s;
    }
}

void orc_search(const uint8_t* cur, const uint8_t* prev, int W, int H, int64_t pitch,
                int B, int R, int kind, int16_t* mv, uint32_t* sse)
{
    orc_search_k(cur, prev, W, H, pitch, B, R, kind, 1, mv, sse);
}

/* Step 3: mean motion of the blocks whose best match passes the PSNR test.
 * out = (Mx, My, K); each mean is rounded to the nearest integer, halves away
 * from zero.  K = 0 gives M = (0, 0). */
void orc_mean_mv(const int16_t* mv, const uint32_t* sse, int W, int H, int B, double T, int32_t* out)
{
    int Gx = (W + B - 1) / B, Gy = (H + B - 1) / B;
    int64_t sx = 0, sy = 0, K = 0;
    for (int b = 0; b < Gx * Gy; ++b) {
        int x0, y0, bw, bh;
        block_geom(W, H, B, b % Gx, b / Gx, &x0, &y0, &bw, &bh);
        if (sse[b] == ORC_NOT_SEARCHED) continue;                 /* skipped by k-skip */
        if (orc_psnr_pass(sse[b], (int64_t)bw * bh * 3, T)) { sx += mv[2 * b]; sy += mv[2 * b + 1]; ++K; }
    }
    out[0] = out[1] = 0; out[2] = (int32_t)K;
    if (K > 0) {
        int64_t ax = sx < 0 ? -sx : sx, ay = sy < 0 ? -sy : sy;
        int64_t mx = (2 * ax + K) / (2 * K), my = (2 * ay + K) / (2 * K);
        out[0] = (int32_t)(sx < 0 ? -mx : mx);
        out[1] = (int32_t)(sy < 0 ? -my : my);
    }
}

/* Step 4: a block is properly matched when the previous-frame block at the
 * global offset M lies inside the frame and passes the PSNR test. */
void orc_verify(const uint8_t* cur, const uint8_t* prev, int W, int H, int64_t pitch, int B,
                int Mx, int My, int K, double T, uint8_t* matched)
{
    int Gx = (W + B - 1) / B, Gy = (H + B - 1) / B;
    for (int b = 0; b < Gx * Gy; ++b) {
        int x0, y0, bw, bh;
        block_geom(W, H, B, b % Gx, b / Gx, &x0, &y0, &bw, &bh);
        matched[b] = 0;
        if (K <= 0) continue;
        uint64_t s = orc_block_sse(cur, prev, W, H, pitch, x0, y0, bw, bh, Mx, My);
        matched[b] = (uint8_t)orc_psnr_pass(s, (int64_t)bw * bh * 3, T);
    }
}

/* Step 5: merge properly matched blocks into rectangles.  Canonical form:
 * maximal horizontal runs in every block row; a run continues the rectangle
 * above it only when the run directly above spans exactly the same columns.
 * Rectangles come out ordered by (y, x) of their top-left corner.  Returns
 * their number; out must hold Gx*Gy entries. */
int orc_merge(const uint8_t* matched, int W, int H, int B, int Mx, int My, orc_region* out)
{
    int Gx = (W + B - 1) / B, Gy = (H + B - 1) / B, n = 0;
    /* open[x0] = index of the rectangle whose latest row has a run starting at x0, with its end */
    int* open_idx = (int*)malloc(sizeof(int) * Gx);
    int* open_end = (int*)malloc(sizeof(int) * Gx);
    int* next_idx = (int*)malloc(sizeof(int) * Gx);
    int* next_end = (int*)malloc(sizeof(int) * Gx);
    for (int i = 0; i < Gx; ++i) open_idx[i] = -1;
    for (int r = 0; r < Gy; ++r) {
        for (int i = 0; i < Gx; ++i) next_idx[i] = -1;
        int c = 0;
        while (c < Gx) {
            if (!matched[r * Gx + c]) { ++c; continue; }
            int c0 = c;
            while (c < Gx && matched[r * Gx + c]) ++c;
            int c1 = c;                                    /* run covers block columns [c0, c1) */
            int y_px = r * B, y_end = (r + 1) * B < H ? (r + 1) * B : H;
            if (open_idx[c0] >= 0 && open_end[c0] == c1) {
                out[open_idx[c0]].h += y_end - y_px;        /* same span above: grow downwards */
                next_idx[c0] = open_idx[c0];
            } else {
                int x_px = c0 * B, x_end = c1 * B < W ? c1 * B : W;
                orc_region g = { x_px, y_px, x_end - x_px, y_end - y_px, x_px + Mx, y_px + My };
                out[n] = g;
                next_idx[c0] = n++;
            }
            next_end[c0] = c1;
        }
        memcpy(open_idx, next_idx, sizeof(int) * Gx);
        memcpy(open_end, next_end, sizeof(int) * Gx);
    }
    free(open_idx); free(open_end); free(next_idx); free(next_end);
    return n;
}

/* Per-block variant of Steps 4-5 (an extension: the paper moves every reused rectangle by the one global
 * vector M; Section 4 notes that this loses blocks that move differently).  Here a searched block is
 * accepted with its OWN best vector when that match passes the PSNR test of Step 2, and Step 5 merges
 * only neighbours that carry the same vector: a horizontal run ends where the vector changes, and a run
 * continues the rectangle above only when that run spans the same columns with the same vector.  Each
 * rectangle's source is its position plus its blocks' vector.  Order and canonical form as orc_merge. */
void orc_accept_own(const int16_t* mv, const uint32_t* sse, int W, int H, int B, double T, uint8_t* matched)
{
    int Gx = (W + B - 1) / B, Gy = (H + B - 1) / B;
    for (int b = 0; b < Gx * Gy; ++b) {
        int x0, y0, bw, bh;
        block_geom(W, H, B, b % Gx, b / Gx, &x0, &y0, &bw, &bh);
        matched[b] = (uint8_t)(sse[b] != ORC_NOT_SEARCHED && orc_psnr_pass(sse[b], (int64_t)bw * bh * 3, T));
    }
}

int orc_merge_own(const uint8_t* matched, const int16_t* mv, int W, int H, int B, orc_region* out)
{
    int Gx = (W + B - 1) / B, Gy = (H + B - 1) / B, n = 0;
    int* open_idx = (int*)malloc(sizeof(int) * Gx);      /* rectangle whose latest row has a run starting here */
    int* open_end = (int*)malloc(sizeof(int) * Gx);
    int* next_idx = (int*)malloc(sizeof(int) * Gx);
    int* next_end = (int*)malloc(sizeof(int) * Gx);
    for (int i = 0; i < Gx; ++i) open_idx[i] = -1;
    for (int r = 0; r < Gy; ++r) {
        for (int i = 0; i < Gx; ++i) next_idx[i] = -1;
        int c = 0;
        while (c < Gx) {
            if (!matched[r * Gx + c]) { ++c; continue; }
            int c0 = c, dx = mv[2 * (r * Gx + c)], dy = mv[2 * (r * Gx + c) + 1];
            while (c < Gx && matched[r * Gx + c] && mv[2 * (r * Gx + c)] == dx && mv[2 * (r * Gx + c) + 1] == dy) ++c;
            int c1 = c;
            int y_px = r * B, y_end = (r + 1) * B < H ? (r + 1) * B : H;
            int up = open_idx[c0];
            if (up >= 0 && open_end[c0] == c1 && out[up].sx - out[up].x == dx && out[up].sy - out[up].y == dy) {
                out[up].h += y_end - y_px;
                next_idx[c0] = up;
            } else {
                int x_px = c0 * B, x_end = c1 * B < W ? c1 * B : W;
                orc_region g = { x_px, y_px, x_end - x_px, y_end - y_px, x_px + dx, y_px + dy };
                out[n] = g;
                next_idx[c0] = n++;
            }
            next_end[c0] = c1;
        }
        memcpy(open_idx, next_idx, sizeof(int) * Gx);
        memcpy(open_end, next_end, sizeof(int) * Gx);
    }
    free(open_idx); free(open_end); free(next_idx); free(next_end);
    return n;
}

/* ------------------------------------------------------------------------
 * Section 5, "Propagation": the region transform D_t of Table 2
 * ---------------------------------------------------------------------- */

static int floor_div(int a, int b) { int q = a / b; return (a % b != 0 && ((a < 0) != (b < 0))) ? q - 1 : q; }
static int ceil_div(int a, int b) { return -floor_div(-a, b); }

/* One axis of a sliding-window layer (convolution, pooling): output o reads
 * inputs [o s - p, o s - p + k - 1]; it is reusable exactly when that whole
 * window lies inside [x, x + w - 1].  First reusable output ceil((x+p)/s)
 * (Table 2), last floor((x + w - k + p)/s): this interval form reproduces the
 * worked examples of Fig. 7 and of Section 4, which the printed width formula
 * misses by one. */
static void erode_axis(int x, int w, int k, int s, int p, int* x_out, int* w_out)
{
    int first = ceil_div(x + p, s);
    int last = floor_div(x + w - k + p, s);
    *x_out = first;
    *w_out = last - first + 1;
}

/* One axis of the area resize n_in -> n_out: output o averages inputs
 * [floor(o n_in / n_out), ceil((o+1) n_in / n_out) - 1]; reusable when that
 * span lies inside [x, x + w - 1]. */
static void resize_axis(int x, int w, int n_in, int n_out, int* x_out, int* w_out)
{
    int first = (int)(((int64_t)x * n_out + n_in - 1) / n_in);           /* ceil(x n_out / n_in) */
    int last = (int)(((int64_t)(x + w) * n_out) / n_in) - 1;             /* floor((x+w) n_out / n_in) - 1 */
    *x_out = first;
    *w_out = last - first + 1;
}

static const orc_region EMPTY_REGION = { 0, 0, 0, 0, 0, 0 };

/* D_t applied to the current-frame rectangle and, independently, to the
 * cached-frame rectangle (Section 5: D_t(x,y,w,h) -> D_t(x',y',w,h)).  When
 * the two results differ in size (motion not a multiple of the stride) the
 * smaller size is kept on each axis. */
static orc_region propagate_window(orc_region r, int kind, int kh, int kw, int sh, int sw, int ph, int pw,
                                   int in_h, int in_w, int out_h, int out_w)
{
    if (r.w <= 0 || r.h <= 0) return EMPTY_REGION;
    int dx, dw, dy, dh, qx, qw, qy, qh;
    if (kind == ORC_RESIZE_AREA) {
        resize_axis(r.x, r.w, in_w, out_w, &dx, &dw);   resize_axis(r.y, r.h, in_h, out_h, &dy, &dh);
        resize_axis(r.sx, r.w, in_w, out_w, &qx, &qw);  resize_axis(r.sy, r.h, in_h, out_h, &qy, &qh);
    } else {
        erode_axis(r.x, r.w, kw, sw, pw, &dx, &dw);     erode_axis(r.y, r.h, kh, sh, ph, &dy, &dh);
        erode_axis(r.sx, r.w, kw, sw, pw, &qx, &qw);    erode_axis(r.sy, r.h, kh, sh, ph, &qy, &qh);
    }
    int w = dw < qw ? dw : qw, h = dh < qh ? dh : qh;
    if (w <= 0 || h <= 0) return EMPTY_REGION;
    orc_region o = { dx, dy, w, h, qx, qy };
    return o;
}

/* Layers with several inputs (Table 2, "Concat": the overlapped region; the
 * residual add is treated the same way): region i survives only when it is
 * present on both inputs with the same displacement between current and
 * cached rectangle; the result is the overlap of the two rectangles. */
static orc_region propagate_overlap(orc_region a, orc_region b)
{
    if (a.w <= 0 || a.h <= 0 || b.w <= 0 || b.h <= 0) return EMPTY_REGION;
    if (a.sx - a.x != b.sx - b.x || a.sy - a.y != b.sy - b.y) return EMPTY_REGION;
    int x0 = a.x > b.x ? a.x : b.x, y0 = a.y > b.y ? a.y : b.y;
    int x1 = (a.x + a.w < b.x + b.w) ? a.x + a.w : b.x + b.w;
    int y1 = (a.y + a.h < b.y + b.h) ? a.y + a.h : b.y + b.h;
    if (x1 <= x0 || y1 <= y0) return EMPTY_REGION;
    orc_region o = { x0, y0, x1 - x0, y1 - y0, x0 + (a.sx - a.x), y0 + (a.sy - a.y) };
    return o;
}

/* One layer of Table 2 applied to n region slots.  Slot i of the output is
 * derived from slot i of the input(s); a region that vanishes becomes the
 * all-zero region and stays in its slot.  in1 is used by add / concat only. */
void orc_propagate_layer(const orc_layer* L, int in_h, int in_w,
                         const orc_region* in0, const orc_region* in1, int n, orc_region* out)
{
    for (int i = 0; i < n; ++i) {
        switch (L->kind) {
        case ORC_CONV: case ORC_MAXPOOL: case ORC_RESIZE_AREA:
            out[i] = propagate_window(in0[i], L->kind, L->kh, L->kw, L->sh, L->sw, L->ph, L->pw,
                                      in_h, in_w, L->out_h, L->out_w);
            break;
        case ORC_LRN: {                    /* Table 2: (x + r, y + r, w - 2r, h - 2r), r = ph */
            orc_region r = in0[i]; int rad = L->ph;
            if (r.w - 2 * rad <= 0 || r.h - 2 * rad <= 0) { out[i] = EMPTY_REGION; break; }
            orc_region o = { r.x + rad, r.y + rad, r.w - 2 * rad, r.h - 2 * rad, r.sx + rad, r.sy + rad };
            out[i] = o;
            break;
        }
        case ORC_ADD: case ORC_CONCAT:
            out[i] = propagate_overlap(in0[i], in1[i]);
            break;
        case ORC_FC:                       /* Table 2: (0, 0, 0, 0) */
            out[i] = EMPTY_REGION;
            break;
        default:                           /* Table 2, "Others": unchanged */
            out[i] = (in0[i].w > 0 && in0[i].h > 0) ? in0[i] : EMPTY_REGION;
            break;
        }
    }
}

/* ------------------------------------------------------------------------
 * Layer arithmetic on double maps
 * ---------------------------------------------------------------------- */

/* Storage rounding.  mode 0: keep the double.  mode 1: round to the nearest
 * bfloat16 (8 significant bits), ties to even. */
double orc_quant(double v, int mode)
{
    if (mode == 0 || v == 0.0 || !isfinite(v)) return v;
    int e = ilogb(v);
    if (e < -126) e = -126;
    return ldexp(nearbyint(ldexp(v, 7 - e)), e - 7);
}

void orc_quant_array(double* v, int64_t n, int mode)
{
    for (int64_t i = 0; i < n; ++i) v[i] = orc_quant(v[i], mode);
}

/* Frame to network input: pixel / 255. */
void orc_input_map(const uint8_t* frame, int W, int H, int64_t pitch, int mode, double* out)
{
    for (int y = 0; y < H; ++y)
        for (int x = 0; x < W * 3; ++x)
            out[(int64_t)y * W * 3 + x] = orc_quant((double)frame[y * pitch + x] / 255.0, mode);
}

/* Area resize of the frame: output (oy, ox) is the mean of the source pixels
 * in rows [floor(oy H/Ho), ceil((oy+1) H/Ho) - 1] and the like columns, / 255. */
void orc_resize_area(const uint8_t* frame, int W, int H, int64_t pitch, int Wo, int Ho, int mode, double* out)
{
    #pragma omp parallel for
    for (int oy = 0; oy < Ho; ++oy)
        for (int ox = 0; ox < Wo; ++ox) {
            int y0 = (int)((int64_t)oy * H / Ho), y1 = (int)(((int64_t)(oy + 1) * H + Ho - 1) / Ho) - 1;
            int x0 = (int)((int64_t)ox * W / Wo), x1 = (int)(((int64_t)(ox + 1) * W + Wo - 1) / Wo) - 1;
            for (int c = 0; c < 3; ++c) {
                int64_t sum = 0;
                for (int y = y0; y <= y1; ++y)
                    for (int x = x0; x <= x1; ++x) sum += frame[y * pitch + x * 3 + c];
                double mean = (double)sum / ((double)((y1 - y0 + 1) * (x1 - x0 + 1)) * 255.0);
                out[((int64_t)oy * Wo + ox) * 3 + c] = orc_quant(mean, mode);
            }
        }
}

/* Section 5, "Reuse": an output pixel inside a reusable rectangle is copied
 * from the cached output of the previous frame at the mapped position; every
 * other pixel is a direct convolution (+ bias, optional ReLU) of the complete
 * input map.  prev_out == NULL or n_regions == 0 is plain full convolution.
 * reused (optional) is a Ho x Wo byte map of which pixels were copied. */
void orc_conv_reuse(const double* in, int Hi, int Wi, const orc_layer* L,
                    const double* weight, const double* bias, int mode,
                    const double* prev_out, const orc_region* regions, int n_regions,
                    double* out, uint8_t* reused)
{
    const int Ho = L->out_h, Wo = L->out_w, Ci = L->cin, Co = L->cout;
    /* grouped convolution (the form the cited AlexNet uses): output channel co of group g = co / (Co / G) sees
     * only the input channels g * Ci / G ... (g + 1) * Ci / G - 1; weights [cout][kh][kw][cin / G] */
    const int G = L->groups > 1 ? L->groups : 1, Cig = Ci / G, Cog = Co / G;
    #pragma omp parallel for schedule(dynamic, 1)
    for (int oy = 0; oy < Ho; ++oy)
        for (int ox = 0; ox < Wo; ++ox) {
            double* o = out + ((int64_t)oy * Wo + ox) * Co;
            int hit = -1;
            if (prev_out)
                for (int r = 0; r < n_regions && hit < 0; ++r)
                    if (ox >= regions[r].x && ox < regions[r].x + regions[r].w &&
                        oy >= regions[r].y && oy < regions[r].y + regions[r].h) hit = r;
            if (reused) reused[oy * Wo + ox] = hit >= 0;
            if (hit >= 0) {
                int py = oy - regions[hit].y + regions[hit].sy, px = ox - regions[hit].x + regions[hit].sx;
                memcpy(o, prev_out + ((int64_t)py * Wo + px) * Co, sizeof(double) * Co);
                continue;
            }
            for (int co = 0; co < Co; ++co) {
                double acc = 0.0;
                for (int ky = 0; ky < L->kh; ++ky) {
                    int iy = oy * L->sh - L->ph + ky;
                    if (iy < 0 || iy >= Hi) continue;
                    for (int kx = 0; kx < L->kw; ++kx) {
                        int ix = ox * L->sw - L->pw + kx;
                        if (ix < 0 || ix >= Wi) continue;
                        const double* a = in + ((int64_t)iy * Wi + ix) * Ci + (co / Cog) * Cig;
                        const double* w = weight + (((int64_t)co * L->kh + ky) * L->kw + kx) * Cig;
                        for (int ci = 0; ci < Cig; ++ci) acc += a[ci] * w[ci];
                    }
                }
                acc += bias[co];
                if (L->relu && acc < 0.0) acc = 0.0;
                o[co] = orc_quant(acc, mode);
            }
        }
}

/* Max pooling, floor mode; window taps outside the map are ignored. */
void orc_maxpool(const double* in, int Hi, int Wi, const orc_layer* L, double* out)
{
    const int Ho = L->out_h, Wo = L->out_w, C = L->cout;
    for (int oy = 0; oy < Ho; ++oy)
        for (int ox = 0; ox < Wo; ++ox)
            for (int c = 0; c < C; ++c) {
                double m = -INFINITY;
                for (int ky = 0; ky < L->kh; ++ky)
                    for (int kx = 0; kx < L->kw; ++kx) {
                        int iy = oy * L->sh - L->ph + ky, ix = ox * L->sw - L->pw + kx;
                        if (iy < 0 || iy >= Hi || ix < 0 || ix >= Wi) continue;
                        double v = in[((int64_t)iy * Wi + ix) * C + c];
                        if (v > m) m = v;
                    }
                out[((int64_t)oy * Wo + ox) * C + c] = m;
            }
}

/* Element-wise sum of two maps, optional ReLU, storage rounding. */
void orc_add(const double* a, const double* b, int64_t n, int relu, int mode, double* out)
{
    for (int64_t i = 0; i < n; ++i) {
        double v = a[i] + b[i];
        if (relu && v < 0.0) v = 0.0;
        out[i] = orc_quant(v, mode);
    }
}

void orc_relu(const double* a, int64_t n, double* out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = a[i] < 0.0 ? 0.0 : a[i];
}
