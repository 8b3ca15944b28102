// C ABI of libdeepcache: cache life cycle and the per-frame driver (declared in deepcache.h).
// Host code only enqueues work; region and tile counts stay on the device.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <new>

#include "dc_common.cuh"

static thread_local char g_last_cuda_error[256];

void dc_note_cuda_error(cudaError_t e, const char* file, int line)
{
    snprintf(g_last_cuda_error, sizeof(g_last_cuda_error), "%s at %s:%d", cudaGetErrorString(e), file, line);
    if (getenv("DC_VERBOSE")) fprintf(stderr, "libdeepcache: CUDA error: %s\n", g_last_cuda_error);
}

void dc_prof_release(dc_cache* c);

void dc_use_match_set(dc_cache* c, int k)
{
    const dc_match_set& m = c->mset[k];
    c->mset_cur = k;
    c->blk_mv = m.blk_mv; c->blk_sse = m.blk_sse; c->matched = m.matched; c->run_end = m.run_end; c->mv_acc = m.mv_acc;
    c->long_list = m.long_list; c->gmv = m.gmv; c->regions0 = m.regions0; c->n_regions = m.n_regions;
}

bool dc_layer_cached(const dc_cache* c, int layer)
{
    const dc_layer_desc& d = c->L[layer].d;
    if (d.kind == DC_CONV) return true;
    return (d.kind == DC_MAXPOOL || d.kind == DC_LRN) && c->cfg.cache_pool && ((size_t)d.cout * c->elt) % 16 == 0;
}

namespace {

// nearest bfloat16 (ties to even) of a double, as its 16 bit pattern
uint16_t bf16_bits_from_double(double v)
{
    if (v == 0.0) return 0;
    int e = ilogb(v);
    if (e < -126) e = -126;
    double q = ldexp(nearbyint(ldexp(v, 7 - e)), e - 7);
    float f = (float)q;                       // exact: q has at most 8 significant bits
    uint32_t u; memcpy(&u, &f, 4);
    return (uint16_t)(u >> 16);
}

template <typename T>
int dev_alloc(dc_cache* c, T** p, size_t count)
{
    size_t bytes = count * sizeof(T);
    if (bytes == 0) bytes = sizeof(T);
    if (cudaMalloc((void**)p, bytes) != cudaSuccess) { cudaGetLastError(); return DC_ERR_ALLOC; }
    c->bytes += bytes;
    return DC_OK;
}
#define DC_TRY(expr) do { int rc__ = (expr); if (rc__ != DC_OK) return rc__; } while (0)

// Can dc_infer_frame run this layer?  LRN needs its window stated consistently, a fully-connected layer must cover
// its whole input map (it then runs as that convolution).
bool layer_executable(const dc_layer_desc& L, int in_h, int in_w)
{
    switch (L.kind) {
    case DC_CONV: case DC_MAXPOOL: case DC_RELU: case DC_ADD: case DC_RESIZE_AREA: case DC_CONCAT: return true;
    case DC_LRN: return L.kh == 2 * L.ph + 1 && L.kw == L.kh && L.pw == L.ph;
    case DC_FC: return L.kh == in_h && L.kw == in_w && L.out_h == 1 && L.out_w == 1;
    default: return false;
    }
}

int validate(const dc_config* cfg, const dc_layer_desc* layers, int n)
{
    if (cfg->channels != 3 || cfg->width < 1 || cfg->height < 1 || cfg->n_streams < 1 || cfg->n_streams > 65535) return DC_ERR_CONFIG;
    if (cfg->block < 4 || cfg->block > 32 || cfg->range < 0 || cfg->range > 64) return DC_ERR_CONFIG;
    if (cfg->search < DC_SEARCH_EXHAUSTIVE || cfg->search > DC_SEARCH_THREE_STEP) return DC_ERR_CONFIG;
    if (cfg->cache_pool != 0 && cfg->cache_pool != 1) return DC_ERR_CONFIG;
    if (cfg->region_mode != DC_REGIONS_GLOBAL && cfg->region_mode != DC_REGIONS_PER_BLOCK) return DC_ERR_CONFIG;
    if (cfg->skip_k < 1 || cfg->skip_k > 16 || cfg->expire_n < 1 || cfg->max_regions < 0) return DC_ERR_CONFIG;
    if (cfg->dtype != DC_FP32 && cfg->dtype != DC_BF16) return DC_ERR_CONFIG;
    if (!(cfg->psnr_db > 0.0) || !(cfg->psnr_db < 200.0)) return DC_ERR_CONFIG;
    if (n < 1 || n > DC_MAX_LAYERS) return DC_ERR_CONFIG;
    const int elt = cfg->dtype == DC_BF16 ? 2 : 4;
    for (int i = 0; i < n; ++i) {
        const dc_layer_desc& L = layers[i];
        if (L.kind < DC_CONV || L.kind > DC_FC) return DC_ERR_CONFIG;
        if (L.in0 < -1 || L.in0 >= i) return DC_ERR_CONFIG;
        int ih = L.in0 < 0 ? cfg->height : layers[L.in0].out_h;
        int iw = L.in0 < 0 ? cfg->width : layers[L.in0].out_w;
        int ic = L.in0 < 0 ? 3 : layers[L.in0].cout;
        if (L.out_h < 1 || L.out_w < 1 || L.cout < 1) return DC_ERR_CONFIG;
        if (L.groups < 0 || (L.groups > 1 && L.kind != DC_CONV)) return DC_ERR_CONFIG;
        switch (L.kind) {
        case DC_CONV: case DC_MAXPOOL:
            if (L.kh < 1 || L.kw < 1 || L.sh < 1 || L.sw < 1 || L.ph < 0 || L.pw < 0) return DC_ERR_CONFIG;
            if (L.ph >= L.kh || L.pw >= L.kw) return DC_ERR_CONFIG;
            if ((ih + 2 * L.ph - L.kh) / L.sh + 1 != L.out_h || (iw + 2 * L.pw - L.kw) / L.sw + 1 != L.out_w) return DC_ERR_CONFIG;
            if (ih + 2 * L.ph < L.kh || iw + 2 * L.pw < L.kw) return DC_ERR_CONFIG;
            if (L.cin != ic) return DC_ERR_CONFIG;
            if (L.kind == DC_CONV && L.groups > 1 && (L.cin % L.groups != 0 || L.cout % L.groups != 0)) return DC_ERR_CONFIG;
            if (L.kind == DC_MAXPOOL && L.cout != ic) return DC_ERR_CONFIG;
            if (L.kind == DC_CONV && (L.cout * elt) % 16 != 0) return DC_ERR_CONFIG;   // 16-byte pixel vectors
            break;
        case DC_ADD: case DC_CONCAT: {
            if (L.in1 < -1 || L.in1 >= i) return DC_ERR_CONFIG;
            int jh = L.in1 < 0 ? cfg->height : layers[L.in1].out_h, jw = L.in1 < 0 ? cfg->width : layers[L.in1].out_w;
            int jc = L.in1 < 0 ? 3 : layers[L.in1].cout;
            if (jh != ih || jw != iw || L.out_h != ih || L.out_w != iw) return DC_ERR_CONFIG;
            if (L.kind == DC_ADD && (jc != ic || L.cout != ic)) return DC_ERR_CONFIG;
            if (L.kind == DC_CONCAT && L.cout != ic + jc) return DC_ERR_CONFIG;
            break;
        }
        case DC_RESIZE_AREA:
            if (L.in0 != -1 || L.cout != 3 || L.out_h > ih || L.out_w > iw) return DC_ERR_CONFIG;
            break;
        case DC_LRN:
            if (L.ph < 0 || L.out_h != ih || L.out_w != iw || L.cout != ic) return DC_ERR_CONFIG;
            break;
        case DC_FC:
            if (L.cin != ic) return DC_ERR_CONFIG;
            if (layer_executable(L, ih, iw) && (L.cout * elt) % 16 != 0) return DC_ERR_CONFIG;
            break;
        case DC_RELU:
            if (L.out_h != ih || L.out_w != iw || L.cout != ic) return DC_ERR_CONFIG;
            break;
        default: break;
        }
    }
    return DC_OK;
}

int build(dc_cache* c, const dc_layer_desc* layers, const void* const* weights_dev, const void* const* bias_dev)
{
    const dc_config& cfg = c->cfg;
    const int S = c->S, n = c->n_layers;
    // cached key frames: own pitch (16-byte multiple, at least 16 spare bytes per row and a spare
    // tail) so the matcher may fetch whole aligned words around any candidate
    c->key_pitch = ((size_t)cfg.width * 3 + 16 + 15) / 16 * 16;
    for (int k = 0; k < 3; ++k) {
        DC_TRY(dev_alloc(c, &c->key[k], c->key_pitch * cfg.height * S + 256));
        DC_CUDA(cudaMemsetAsync(c->key[k], 0, c->key_pitch * cfg.height * S + 256, c->stream));
    }
    {
        int dev = 0, sms = 148;
        DC_CUDA(cudaGetDevice(&dev));
        DC_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        c->num_sms = sms;
        c->device = dev;
    }
    const size_t nblk = (size_t)S * c->Gx * c->Gy;
    for (int k = 0; k < 2; ++k) {
        dc_match_set& m = c->mset[k];
        DC_TRY(dev_alloc(c, &m.blk_mv, nblk * 2));
        DC_TRY(dev_alloc(c, &m.blk_sse, nblk));
        DC_TRY(dev_alloc(c, &m.matched, nblk));
        DC_TRY(dev_alloc(c, &m.run_end, nblk));
        DC_TRY(dev_alloc(c, &m.mv_acc, (size_t)S * 4 + 4));
        DC_TRY(dev_alloc(c, &m.long_list, nblk));
        DC_TRY(dev_alloc(c, &m.gmv, (size_t)S * 3));
        DC_TRY(dev_alloc(c, &m.regions0, (size_t)S * c->max_regions));
        DC_TRY(dev_alloc(c, &m.n_regions, (size_t)S));
        DC_CUDA(cudaMemsetAsync(m.n_regions, 0, sizeof(int32_t) * S, c->stream));
    }
    dc_use_match_set(c, 0);
    DC_TRY(dev_alloc(c, &c->table, (size_t)n * S * c->max_regions));
    DC_TRY(dev_alloc(c, &c->layers_dev, (size_t)n));
    DC_TRY(dev_alloc(c, &c->in_hw_dev, (size_t)n * 2));
    DC_TRY(dev_alloc(c, &c->dirty_count, (size_t)n));
    DC_TRY(dev_alloc(c, &c->all_count, (size_t)n * 2));
    DC_TRY(dev_alloc(c, &c->reuse_px, (size_t)n * S * 2));
    c->alive = c->reuse_px + (size_t)n * S;
    DC_TRY(dev_alloc(c, &c->status, (size_t)1));
    DC_TRY(dev_alloc(c, &c->reused_total, (size_t)n));
    DC_CUDA(cudaMemsetAsync(c->reused_total, 0, sizeof(unsigned long long) * n, c->stream));
    DC_CUDA(cudaMemsetAsync(c->status, 0, sizeof(int32_t), c->stream));
    DC_CUDA(cudaMemsetAsync(c->table, 0, sizeof(dc_region) * n * S * c->max_regions, c->stream));
    DC_CUDA(cudaMemcpyAsync(c->layers_dev, layers, sizeof(dc_layer_desc) * n, cudaMemcpyHostToDevice, c->stream));

    // PSNR > T as an integer bound on the SSE, for the four block shapes of a clipped grid
    for (int i = 0; i < 4; ++i) {
        int bw = (i & 1) ? cfg.width - (c->Gx - 1) * cfg.block : cfg.block;
        int bh = (i & 2) ? cfg.height - (c->Gy - 1) * cfg.block : cfg.block;
        double q = 65025.0 * (double)(bw * bh * 3) / pow(10.0, cfg.psnr_db / 10.0);
        double lim = ceil(q) - 1.0;
        c->sse_limit[i] = lim >= 4294967295.0 ? 4294967295u : (uint32_t)lim;
    }
    // pixel -> map element table
    if (cfg.dtype == DC_BF16) {
        uint16_t lut[256];
        for (int i = 0; i < 256; ++i) lut[i] = bf16_bits_from_double((double)i / 255.0);
        DC_TRY(dev_alloc(c, (uint16_t**)&c->pix_lut, (size_t)256));
        DC_CUDA(cudaMemcpy(c->pix_lut, lut, sizeof(lut), cudaMemcpyHostToDevice));
    } else {
        float lut[256];
        for (int i = 0; i < 256; ++i) lut[i] = (float)((double)i / 255.0);
        DC_TRY(dev_alloc(c, (float**)&c->pix_lut, (size_t)256));
        DC_CUDA(cudaMemcpy(c->pix_lut, lut, sizeof(lut), cudaMemcpyHostToDevice));
    }

    int32_t in_hw[DC_MAX_LAYERS * 2], all_count[DC_MAX_LAYERS * 2];
    size_t max_tiles = 1;
    bool need_input_map = false;
    for (int i = 0; i < n; ++i) {
        dc_layer_rt& L = c->L[i];
        L.d = layers[i];
        // an executable fully-connected layer runs as the convolution that covers its input map; the device copy of the
        // layer table keeps DC_FC, so Table 2 still marks nothing of its output reusable and every tile is computed
        if (L.d.kind == DC_FC && c->executable) { L.d.kind = DC_CONV; L.d.sh = L.d.sw = 1; L.d.ph = L.d.pw = 0; }
        L.in_h = L.d.in0 < 0 ? cfg.height : layers[L.d.in0].out_h;
        L.in_w = L.d.in0 < 0 ? cfg.width : layers[L.d.in0].out_w;
        in_hw[2 * i] = L.in_h; in_hw[2 * i + 1] = L.in_w;
        all_count[i] = 0; all_count[n + i] = 0;
        if (!c->executable) continue;
        if (L.d.in0 < 0 && L.d.kind != DC_RESIZE_AREA) need_input_map = true;
        if ((L.d.kind == DC_ADD || L.d.kind == DC_CONCAT) && L.d.in1 < 0) need_input_map = true;
        L.map_bytes = (size_t)S * L.d.out_h * L.d.out_w * L.d.cout * c->elt;
        const bool cached = dc_layer_cached(c, i);
        const int copies = cached ? 2 : 1;
        for (int k = 0; k < copies; ++k) {
            DC_TRY(dev_alloc(c, (uint8_t**)&L.map[k], L.map_bytes));
            DC_CUDA(cudaMemsetAsync(L.map[k], 0, L.map_bytes, c->stream));
        }
        if (cached) {
            L.tiles_x = dc_div_up(L.d.out_w, DC_TILE_W);
            L.tiles_y = dc_div_up(L.d.out_h, DC_TILE_H);
            L.gpr = dc_div_up(L.d.out_w, DC_TILE_W);
            L.tiles_flat = (int)(((size_t)S * L.d.out_h * L.gpr + DC_TILE_H - 1) / DC_TILE_H);
            size_t tiles = (size_t)L.tiles_x * L.tiles_y * S;             // never fewer than the flat tiles
            if (tiles > max_tiles) max_tiles = tiles;
            all_count[i] = (int32_t)tiles; all_count[n + i] = L.tiles_flat;
            DC_TRY(dev_alloc(c, &L.masks, tiles * 4));
            DC_TRY(dev_alloc(c, &L.dirty_list, tiles));
            DC_TRY(dev_alloc(c, &L.all_list, tiles));
            int32_t* iota = (int32_t*)malloc(sizeof(int32_t) * tiles);
            if (!iota) return DC_ERR_ALLOC;
            for (size_t t = 0; t < tiles; ++t) iota[t] = (int32_t)t;
            cudaError_t e = cudaMemcpy(L.all_list, iota, sizeof(int32_t) * tiles, cudaMemcpyHostToDevice);
            free(iota);
            DC_CUDA(e);
        }
        if (L.d.kind == DC_CONV) {
            if (!weights_dev || !bias_dev || !weights_dev[i] || !bias_dev[i]) return DC_ERR_ARG;
            DC_TRY(dc_pack_weights(c, i, (const float*)weights_dev[i], (const float*)bias_dev[i]));
        }
    }
    DC_CUDA(cudaMemcpyAsync(c->in_hw_dev, in_hw, sizeof(int32_t) * 2 * n, cudaMemcpyHostToDevice, c->stream));
    DC_CUDA(cudaMemcpyAsync(c->all_count, all_count, sizeof(int32_t) * 2 * n, cudaMemcpyHostToDevice, c->stream));
    DC_TRY(dev_alloc(c, &c->zero_masks, max_tiles * 4));
    DC_CUDA(cudaMemsetAsync(c->zero_masks, 0, max_tiles * 4 * sizeof(uint32_t), c->stream));
    if (need_input_map)
        DC_TRY(dev_alloc(c, (uint8_t**)&c->input_map, (size_t)S * cfg.height * cfg.width * 3 * c->elt));
    size_t stat_ints = (size_t)S * (3 + 4 + 1) + (size_t)n * S;
    if (cudaMallocHost(&c->stats_pinned, stat_ints * sizeof(int32_t)) != cudaSuccess) { cudaGetLastError(); return DC_ERR_ALLOC; }
    DC_CUDA(cudaStreamSynchronize(c->stream));      // layers / in_hw / all_count live on this stack frame
    for (int i = 0; i < n; ++i)
        if (c->executable && c->L[i].d.kind == DC_CONV) {
            const void* in = c->L[i].d.in0 < 0 ? c->input_map : c->L[c->L[i].d.in0].map[0];
            if (c->L[i].s2d_s) in = c->L[i].in_s2d;               // the kernels being timed read the block map
            DC_TRY(dc_conv_bf16_autotune(c, i, in));
        }
    if (c->executable) DC_TRY(dc_build_classify_table(c));       // after the tuner: it decides each layer's tile geometry
    DC_CUDA(cudaStreamSynchronize(c->stream));
    return DC_OK;
}

void release(dc_cache* c)
{
    dc_prof_release(c);
    cudaFree(c->reused_total);
    if (c->la_stream) { cudaStreamSynchronize(c->la_stream); cudaEventDestroy(c->ev_key); cudaEventDestroy(c->ev_match); cudaStreamDestroy(c->la_stream); }
    if (c->copy_stream) { cudaStreamSynchronize(c->copy_stream); cudaEventDestroy(c->copied[0]); cudaEventDestroy(c->copied[1]); cudaStreamDestroy(c->copy_stream); }
    for (int k = 0; k < 3; ++k) cudaFree(c->key[k]);
    cudaFree(c->staging[0]); cudaFree(c->staging[1]);
    for (int k = 0; k < 2; ++k) {
        dc_match_set& m = c->mset[k];
        cudaFree(m.blk_mv); cudaFree(m.blk_sse); cudaFree(m.matched); cudaFree(m.run_end); cudaFree(m.mv_acc);
        cudaFree(m.long_list); cudaFree(m.gmv); cudaFree(m.regions0); cudaFree(m.n_regions);
    }
    cudaFree(c->table); cudaFree(c->classify_table);
    cudaFree(c->layers_dev); cudaFree(c->in_hw_dev); cudaFree(c->dirty_count); cudaFree(c->all_count);
    cudaFree(c->reuse_px); cudaFree(c->zero_masks); cudaFree(c->status); cudaFree(c->input_map); cudaFree(c->pix_lut);
    if (c->stats_pinned) cudaFreeHost(c->stats_pinned);
    for (int i = 0; i < c->n_layers; ++i) {
        dc_layer_rt& L = c->L[i];
        cudaFree(L.map[0]); cudaFree(L.map[1]); cudaFree(L.weight); cudaFree(L.bias); cudaFree(L.weight_packed); cudaFree(L.in_padded); cudaFree(L.in_s2d); cudaFree(L.weight_halo);
        cudaFree(L.masks); cudaFree(L.dirty_list); cudaFree(L.all_list);
    }
    cudaGetLastError();
    delete c;
}

const void* layer_input(dc_cache* c, int idx)
{
    if (idx < 0) return c->input_map;
    dc_layer_rt& P = c->L[idx];
    return P.map[dc_layer_cached(c, idx) ? P.cur : 0];
}

// Drops a pending lookahead: the main stream first waits for it, so nothing it wrote is still in flight.
int cancel_lookahead(dc_cache* c)
{
    if (c->la_frame) {
        DC_CUDA(cudaStreamWaitEvent(c->stream, c->ev_match, 0));
        c->la_frame = nullptr;
    }
    return DC_OK;
}

int fill_stats(dc_cache* c, bool refreshed, dc_frame_stats* stats)
{
    const int S = c->S, n = c->n_layers;
    int32_t* h = (int32_t*)c->stats_pinned;
    int32_t* h_gmv = h; int32_t* h_acc = h + 3 * S; int32_t* h_nreg = h + 7 * S; int32_t* h_reuse = h + 8 * S;
    if (!refreshed) {
        DC_CUDA(cudaMemcpyAsync(h_gmv, c->gmv, sizeof(int32_t) * 3 * S, cudaMemcpyDeviceToHost, c->stream));
        DC_CUDA(cudaMemcpyAsync(h_acc, c->mv_acc, sizeof(int32_t) * 4 * S, cudaMemcpyDeviceToHost, c->stream));
        DC_CUDA(cudaMemcpyAsync(h_nreg, c->n_regions, sizeof(int32_t) * S, cudaMemcpyDeviceToHost, c->stream));
        DC_CUDA(cudaMemcpyAsync(h_reuse, c->reuse_px, sizeof(int32_t) * n * S, cudaMemcpyDeviceToHost, c->stream));
    }
    DC_CUDA(cudaStreamSynchronize(c->stream));
    for (int s = 0; s < S; ++s) {
        dc_frame_stats& st = stats[s];
        memset(&st, 0, sizeof(st));
        st.refreshed = refreshed ? 1 : 0;
        st.n_blocks = c->Gx * c->Gy;
        if (refreshed) continue;
        st.mvx = h_gmv[3 * s]; st.mvy = h_gmv[3 * s + 1]; st.k_passed = h_gmv[3 * s + 2];
        st.n_matched = h_acc[4 * s + 3]; st.n_regions = h_nreg[s];
        for (int l = 0; l < n; ++l)
            if (dc_layer_cached(c, l))
                st.reuse_ratio[l] = (float)h_reuse[(size_t)l * S + s] / (float)(c->L[l].d.out_h * c->L[l].d.out_w);
    }
    return DC_OK;
}

}  // namespace

extern "C" {

int dc_cache_create(const dc_config* cfg, const dc_layer_desc* layers, int n_layers,
                    const void* const* weights_dev, const void* const* bias_dev, void* cuda_stream, dc_cache** out)
{
    if (!cfg || !layers || !out) return DC_ERR_ARG;
    *out = nullptr;
    int rc = validate(cfg, layers, n_layers);
    if (rc != DC_OK) return rc;
    dc_cache* c = new (std::nothrow) dc_cache();
    if (!c) return DC_ERR_ALLOC;
    memset((void*)c, 0, sizeof(*c));
    c->cfg = *cfg; c->n_layers = n_layers; c->stream = (cudaStream_t)cuda_stream;
    c->S = cfg->n_streams;
    c->Gx = dc_div_up(cfg->width, cfg->block); c->Gy = dc_div_up(cfg->height, cfg->block);
    // Step 5 never yields more than ceil(Gx / 2) * Gy rectangles (runs in a row are separated)
    // worst case: alternating matched / unmatched blocks in every row; in per-block mode every block on its own
    const int worst = cfg->region_mode == DC_REGIONS_PER_BLOCK ? c->Gx * c->Gy : dc_div_up(c->Gx, 2) * c->Gy;
    c->max_regions = cfg->max_regions > 0 ? cfg->max_regions : worst;
    c->elt = cfg->dtype == DC_BF16 ? 2 : 4;
    c->executable = true;
    for (int i = 0; i < n_layers; ++i) {
        const int ih = layers[i].in0 < 0 ? cfg->height : layers[layers[i].in0].out_h;
        const int iw = layers[i].in0 < 0 ? cfg->width : layers[layers[i].in0].out_w;
        if (!layer_executable(layers[i], ih, iw)) c->executable = false;
    }
    rc = build(c, layers, weights_dev, bias_dev);
    if (rc != DC_OK) { release(c); return rc; }
    *out = c;
    return DC_OK;
}

int dc_cache_destroy(dc_cache* c)
{
    if (!c) return DC_ERR_ARG;
    cudaStreamSynchronize(c->stream);
    release(c);
    return DC_OK;
}

int dc_cache_reset(dc_cache* c)
{
    if (!c) return DC_ERR_ARG;
    DC_TRY(cancel_lookahead(c));
    c->key_valid = false; c->frame_idx = 0; c->frames_cached = 0; c->frames_full = 0;
    DC_CUDA(cudaMemsetAsync(c->status, 0, sizeof(int32_t), c->stream));
    DC_CUDA(cudaMemsetAsync(c->reused_total, 0, sizeof(unsigned long long) * c->n_layers, c->stream));
    return DC_OK;
}

int dc_cache_bytes(const dc_cache* c, size_t* bytes)
{
    if (!c || !bytes) return DC_ERR_ARG;
    *bytes = c->bytes;
    return DC_OK;
}

int dc_cache_launches(const dc_cache* c, int64_t* launches)
{
    if (!c || !launches) return DC_ERR_ARG;
    *launches = c->launches;
    return DC_OK;
}

int dc_cache_set_key(dc_cache* c, const uint8_t* frame_dev, size_t pitch)
{
    if (!c || !frame_dev || pitch < (size_t)c->cfg.width * 3) return DC_ERR_ARG;
    DC_TRY(cancel_lookahead(c));
    DC_TRY(dc_launch_copy_frame(c, frame_dev, pitch, c->key[c->key_cur]));
    c->key_valid = true;
    return DC_OK;
}

int dc_match_blocks(dc_cache* c, const uint8_t* frame_dev, size_t pitch, int16_t* block_mv_dev,
                    uint32_t* block_sse_dev, uint8_t* matched_dev, int32_t* global_mv_dev,
                    dc_region* regions_dev, int32_t* n_regions_dev)
{
    if (!c || !frame_dev || pitch < (size_t)c->cfg.width * 3) return DC_ERR_ARG;
    if (!c->key_valid) return DC_ERR_STATE;
    DC_TRY(cancel_lookahead(c));
    uint8_t* scratch = c->key[(c->key_cur + 1) % 3];                             // scratch copy; the cache key stays
    DC_TRY(dc_launch_copy_frame(c, frame_dev, pitch, scratch));
    DC_TRY(dc_launch_match(c, scratch, c->key[c->key_cur]));
    const size_t nblk = (size_t)c->S * c->Gx * c->Gy;
    const cudaMemcpyKind k = cudaMemcpyDeviceToDevice;
    if (block_mv_dev) DC_CUDA(cudaMemcpyAsync(block_mv_dev, c->blk_mv, nblk * 2 * sizeof(int16_t), k, c->stream));
    if (block_sse_dev) DC_CUDA(cudaMemcpyAsync(block_sse_dev, c->blk_sse, nblk * sizeof(uint32_t), k, c->stream));
    if (matched_dev) DC_CUDA(cudaMemcpyAsync(matched_dev, c->matched, nblk, k, c->stream));
    if (global_mv_dev) DC_CUDA(cudaMemcpyAsync(global_mv_dev, c->gmv, sizeof(int32_t) * 3 * c->S, k, c->stream));
    if (regions_dev) DC_CUDA(cudaMemcpyAsync(regions_dev, c->regions0, sizeof(dc_region) * c->S * c->max_regions, k, c->stream));
    if (n_regions_dev) DC_CUDA(cudaMemcpyAsync(n_regions_dev, c->n_regions, sizeof(int32_t) * c->S, k, c->stream));
    return DC_OK;
}

int dc_propagate_regions(dc_cache* c, const dc_region* in_dev, const int32_t* n_in_dev, int layer_begin,
                         int layer_end, dc_region* out_dev, int32_t* n_out_dev)
{
    if (!c || !in_dev || !n_in_dev || !out_dev) return DC_ERR_ARG;
    if (layer_begin < 0 || layer_end > c->n_layers || layer_begin >= layer_end) return DC_ERR_ARG;
    const size_t per_layer = (size_t)c->S * c->max_regions;
    // slots beyond n_in keep whatever an earlier call left: clear the table first
    DC_CUDA(cudaMemsetAsync(c->table, 0, sizeof(dc_region) * per_layer * layer_end, c->stream));
    DC_CUDA(cudaMemsetAsync(c->alive, 0, sizeof(int32_t) * c->n_layers * c->S, c->stream));
    DC_TRY(dc_launch_propagate(c, in_dev, n_in_dev, layer_end));
    DC_CUDA(cudaMemcpyAsync(out_dev, c->table + per_layer * layer_begin,
                            sizeof(dc_region) * per_layer * (layer_end - layer_begin), cudaMemcpyDeviceToDevice, c->stream));
    if (n_out_dev)
        for (int l = 0; l < layer_end - layer_begin; ++l)
            DC_CUDA(cudaMemcpyAsync(n_out_dev + (size_t)l * c->S, n_in_dev, sizeof(int32_t) * c->S,
                                    cudaMemcpyDeviceToDevice, c->stream));
    return DC_OK;
}

int dc_conv_partial(dc_cache* c, int layer, const void* in_map_dev, const void* prev_out_dev,
                    const dc_region* regions_dev, const int32_t* n_regions_dev, void* out_map_dev)
{
    if (!c || !in_map_dev || !out_map_dev || layer < 0 || layer >= c->n_layers) return DC_ERR_ARG;
    if (!c->executable || c->L[layer].d.kind != DC_CONV) return DC_ERR_CONFIG;
    dc_layer_rt& L = c->L[layer];
    const int tiles = dc_layer_tiles(c, L);
    if (regions_dev || n_regions_dev) {
        if (!regions_dev || !n_regions_dev || !prev_out_dev || prev_out_dev == out_map_dev) return DC_ERR_ARG;
        DC_CUDA(cudaMemsetAsync(c->dirty_count + layer, 0, sizeof(int32_t), c->stream));
        DC_CUDA(cudaMemsetAsync(c->reuse_px + (size_t)layer * c->S, 0, sizeof(int32_t) * c->S, c->stream));
        DC_TRY(dc_launch_classify_copy(c, layer, regions_dev, n_regions_dev, prev_out_dev, out_map_dev));
        return dc_launch_conv(c, layer, in_map_dev, out_map_dev, L.dirty_list, c->dirty_count + layer, L.masks, tiles);
    }
    return dc_launch_conv(c, layer, in_map_dev, out_map_dev, L.all_list, dc_all_count(c, layer), c->zero_masks, tiles);
}

int dc_infer_frame(dc_cache* c, const uint8_t* frame_dev, size_t pitch, void* out_map_dev, dc_frame_stats* stats)
{
    if (!c || !frame_dev || pitch < (size_t)c->cfg.width * 3) return DC_ERR_ARG;
    if (!c->executable) return DC_ERR_STATE;
    const int n = c->n_layers, S = c->S;
    // Section 5: the cache is dropped and a whole new frame computed every N frames
    const bool refresh = !c->key_valid || (c->frame_idx % c->cfg.expire_n) == 0;
    // the library's own aligned copy of the frame: matched now, the cache key of the next frame (Section 3)
    uint8_t* frame_copy = c->key[(c->key_cur + 1) % 3];
    const bool looked_ahead = c->la_frame == frame_dev && c->la_pitch == pitch && c->key_valid;
    c->overlap_mode = looked_ahead;                   // a caller that looks ahead keeps doing so: see ring_budget()
    if (looked_ahead) {
        // dc_lookahead_frame already copied this frame in and (unless it is a full frame) matched it
        DC_CUDA(cudaStreamWaitEvent(c->stream, c->ev_match, 0));
        c->la_frame = nullptr;
    } else {
        DC_TRY(cancel_lookahead(c));
        DC_TRY(dc_launch_copy_frame(c, frame_dev, pitch, frame_copy));
    }
    if (c->la_stream) DC_CUDA(cudaEventRecord(c->ev_key, c->stream));   // a later lookahead may start from here
    if (!refresh) {
        DC_CUDA(cudaMemsetAsync(c->dirty_count, 0, sizeof(int32_t) * n, c->stream));
        DC_CUDA(cudaMemsetAsync(c->reuse_px, 0, sizeof(int32_t) * n * S * 2, c->stream));     // and `alive` behind it
        if (looked_ahead && c->la_matched) dc_use_match_set(c, c->mset_cur ^ 1);              // results are waiting there
        else DC_TRY(dc_launch_match(c, frame_copy, c->key[c->key_cur]));
        DC_TRY(dc_launch_propagate(c, c->regions0, c->n_regions, n));
    }
    if (c->input_map) DC_TRY(dc_launch_input_map(c, frame_copy, c->key_pitch));
    const size_t per_layer = (size_t)S * c->max_regions;
    // bitmaps, reuse copies and dirty lists of every cached layer in one launch (they need only the rectangles and
    // each layer's own cached map); possible while all cached layers keep their newest map at the same index
    bool classified = false;
    if (!refresh && c->n_cached > 0) {
        int cur = -1; bool same = true;
        for (int i = 0; i < n; ++i)
            if (dc_layer_cached(c, i)) { if (cur < 0) cur = c->L[i].cur; else if (c->L[i].cur != cur) same = false; }
        if (same) { DC_TRY(dc_launch_classify_all(c, cur)); classified = true; }
    }
    for (int i = 0; i < n; ++i) {
        dc_layer_rt& L = c->L[i];
        const void* in = layer_input(c, L.d.in0);
        switch (L.d.kind) {
        case DC_CONV: {
            const int tiles = dc_layer_tiles(c, L);
            void* prev = L.map[L.cur]; void* out = L.map[L.cur ^ 1];
            if (!refresh) {
                if (!classified) DC_TRY(dc_launch_classify_copy(c, i, c->table + per_layer * i, c->n_regions, prev, out));
                DC_TRY(dc_launch_conv(c, i, in, out, L.dirty_list, c->dirty_count + i, L.masks, tiles));
            } else {
                DC_TRY(dc_launch_conv(c, i, in, out, L.all_list, dc_all_count(c, i), c->zero_masks, tiles));
            }
            L.cur ^= 1;          // the newest output is next frame's cached value
            break;
        }
        case DC_MAXPOOL: {
            if (!dc_layer_cached(c, i)) { DC_TRY(dc_launch_maxpool(c, i, in, L.map[0], nullptr)); break; }
            void* prev = L.map[L.cur]; void* out = L.map[L.cur ^ 1];
            if (!refresh) {           // Section 5's three steps on a pooling layer: copy, mark, compute the rest
                if (!classified) DC_TRY(dc_launch_classify_copy(c, i, c->table + per_layer * i, c->n_regions, prev, out));
                DC_TRY(dc_launch_maxpool(c, i, in, out, L.masks));
            } else {
                DC_TRY(dc_launch_maxpool(c, i, in, out, nullptr));
            }
            L.cur ^= 1;
            break;
        }
        case DC_ADD: DC_TRY(dc_launch_add(c, i, in, layer_input(c, L.d.in1))); break;
        case DC_RELU: DC_TRY(dc_launch_relu(c, i, in)); break;
        case DC_LRN: {
            if (!dc_layer_cached(c, i)) { DC_TRY(dc_launch_lrn(c, i, in, L.map[0], nullptr)); break; }
            void* prev = L.map[L.cur]; void* out = L.map[L.cur ^ 1];
            if (!refresh) {
                if (!classified) DC_TRY(dc_launch_classify_copy(c, i, c->table + per_layer * i, c->n_regions, prev, out));
                DC_TRY(dc_launch_lrn(c, i, in, out, L.masks));
            } else {
                DC_TRY(dc_launch_lrn(c, i, in, out, nullptr));
            }
            L.cur ^= 1;
            break;
        }
        case DC_CONCAT: {
            const int ca = L.d.in0 < 0 ? 3 : c->L[L.d.in0].d.cout, cb = L.d.in1 < 0 ? 3 : c->L[L.d.in1].d.cout;
            DC_TRY(dc_launch_concat(c, i, in, ca, layer_input(c, L.d.in1), cb));
            break;
        }
        case DC_RESIZE_AREA: DC_TRY(dc_launch_resize(c, i, frame_copy, c->key_pitch)); break;
        default: return DC_ERR_STATE;
        }
    }
    c->key_cur = (c->key_cur + 1) % 3;      // the frame becomes the next cache key
    c->key_valid = true;
    c->frame_idx += 1;
    if (refresh) c->frames_full += 1; else c->frames_cached += 1;
    c->last_refreshed = refresh;
    if (out_map_dev)
        DC_CUDA(cudaMemcpyAsync(out_map_dev, layer_input(c, n - 1), c->L[n - 1].map_bytes, cudaMemcpyDeviceToDevice, c->stream));
    if (stats) return fill_stats(c, refresh, stats);
    return DC_OK;
}

static int ensure_lookahead_stream(dc_cache* c)
{
    if (c->la_stream) return DC_OK;
    int least = 0, greatest = 0;
    DC_CUDA(cudaDeviceGetStreamPriorityRange(&least, &greatest));
    DC_CUDA(cudaStreamCreateWithPriority(&c->la_stream, cudaStreamNonBlocking, least));
    DC_CUDA(cudaEventCreateWithFlags(&c->ev_key, cudaEventDisableTiming));
    DC_CUDA(cudaEventCreateWithFlags(&c->ev_match, cudaEventDisableTiming));
    DC_CUDA(cudaEventRecord(c->ev_key, c->stream));     // first use: everything enqueued so far
    return DC_OK;
}

int dc_lookahead_frame(dc_cache* c, const uint8_t* frame_dev, size_t pitch)
{
    if (!c || !frame_dev || pitch < (size_t)c->cfg.width * 3) return DC_ERR_ARG;
    if (!c->executable || !c->key_valid) return DC_ERR_STATE;       // needs a frame to match against
    DC_TRY(ensure_lookahead_stream(c));
    DC_TRY(cancel_lookahead(c));
    // Everything the side stream touches is free once the main stream has passed the frame copy of the last
    // dc_infer_frame (where ev_key was recorded): the third key buffer was last read two frames ago, and the
    // match set that the current inference does not read was last read by the frame before it.  Waiting for
    // that point only -- not for the end of the current inference -- is what lets the two overlap.
    DC_CUDA(cudaStreamWaitEvent(c->la_stream, c->ev_key, 0));
    const bool next_is_full = (c->frame_idx % c->cfg.expire_n) == 0;
    cudaStream_t main_stream = c->stream;
    const int main_set = c->mset_cur;
    c->stream = c->la_stream;                                       // the launchers enqueue on c->stream
    uint8_t* next_copy = c->key[(c->key_cur + 1) % 3];
    int rc = dc_launch_copy_frame(c, frame_dev, pitch, next_copy);
    if (rc == DC_OK && !next_is_full) {
        dc_use_match_set(c, main_set ^ 1);
        rc = dc_launch_match(c, next_copy, c->key[c->key_cur]);
        dc_use_match_set(c, main_set);
    }
    c->stream = main_stream;
    if (rc != DC_OK) return rc;
    DC_CUDA(cudaEventRecord(c->ev_match, c->la_stream));
    c->la_frame = frame_dev; c->la_pitch = pitch; c->la_matched = !next_is_full;
    return DC_OK;
}

static int ensure_staging(dc_cache* c, size_t bytes)
{
    for (int k = 0; k < 2; ++k)
        if (!c->staging[k]) {
            if (cudaMalloc((void**)&c->staging[k], bytes + 256) != cudaSuccess) { cudaGetLastError(); return DC_ERR_ALLOC; }
            c->bytes += bytes + 256;
        }
    return DC_OK;
}

int dc_prefetch_frame_host(dc_cache* c, const uint8_t* frame_host, size_t pitch)
{
    if (!c || !frame_host || pitch < (size_t)c->cfg.width * 3) return DC_ERR_ARG;
    const size_t bytes = pitch * (size_t)c->cfg.height * c->S;
    DC_TRY(ensure_staging(c, bytes));
    if (!c->copy_stream) {
        DC_CUDA(cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking));
        for (int k = 0; k < 2; ++k) DC_CUDA(cudaEventCreateWithFlags(&c->copied[k], cudaEventDisableTiming));
    }
    // a staging buffer that holds no pending prefetch; dc_infer_frame_host waits for its own work before it
    // returns, so such a buffer is idle
    int slot = -1;
    for (int k = 0; k < 2; ++k) if (!c->prefetched[k]) { slot = k; break; }
    if (slot < 0) return DC_ERR_STATE;                           // two frames are already on their way
    DC_CUDA(cudaMemcpyAsync(c->staging[slot], frame_host, bytes, cudaMemcpyHostToDevice, c->copy_stream));
    DC_CUDA(cudaEventRecord(c->copied[slot], c->copy_stream));
    c->prefetched[slot] = frame_host; c->prefetched_pitch[slot] = pitch;
    return DC_OK;
}

int dc_infer_frame_host(dc_cache* c, const uint8_t* frame_host, size_t pitch, void* out_map_host, dc_frame_stats* stats)
{
    if (!c || !frame_host || pitch < (size_t)c->cfg.width * 3) return DC_ERR_ARG;
    const size_t bytes = pitch * (size_t)c->cfg.height * c->S;
    DC_TRY(ensure_staging(c, bytes));
    int slot = -1;
    for (int k = 0; k < 2; ++k)
        if (c->prefetched[k] == frame_host && c->prefetched_pitch[k] == pitch) slot = k;
    if (slot >= 0) {
        DC_CUDA(cudaStreamWaitEvent(c->stream, c->copied[slot], 0));     // the copy is already on its way
    } else {
        for (int k = 0; k < 2; ++k) if (!c->prefetched[k]) { slot = k; break; }
        if (slot < 0) {                                           // both buffers hold prefetches of other frames: drop one
            DC_CUDA(cudaStreamSynchronize(c->copy_stream));
            slot = 0;
        }
        DC_CUDA(cudaMemcpyAsync(c->staging[slot], frame_host, bytes, cudaMemcpyHostToDevice, c->stream));
    }
    c->prefetched[slot] = nullptr;
    int rc = dc_infer_frame(c, c->staging[slot], pitch, nullptr, nullptr);
    if (rc != DC_OK) return rc;
    // a frame that is already prefetched can be matched on the side stream while this one is computed
    const int other = slot ^ 1;
    if (c->prefetched[other] && c->prefetched_pitch[other] == pitch && c->executable) {
        DC_TRY(ensure_lookahead_stream(c));
        DC_CUDA(cudaStreamWaitEvent(c->la_stream, c->copied[other], 0));
        rc = dc_lookahead_frame(c, c->staging[other], pitch);
        if (rc != DC_OK) return rc;
    }
    if (stats) { rc = fill_stats(c, c->last_refreshed, stats); if (rc != DC_OK) return rc; }
    if (out_map_host)
        DC_CUDA(cudaMemcpyAsync(out_map_host, layer_input(c, c->n_layers - 1), c->L[c->n_layers - 1].map_bytes,
                                cudaMemcpyDeviceToHost, c->stream));
    DC_CUDA(cudaStreamSynchronize(c->stream));
    return DC_OK;
}

int dc_cache_layer_map(dc_cache* c, int layer, void** map_dev, size_t* bytes)
{
    if (!c || layer < 0 || layer >= c->n_layers || !map_dev || !c->executable) return DC_ERR_ARG;
    *map_dev = (void*)layer_input(c, layer);
    if (bytes) *bytes = c->L[layer].map_bytes;
    return DC_OK;
}

int dc_cache_layer_conv_scheme(const dc_cache* c, int layer, int32_t* scheme)
{
    if (!c || layer < 0 || layer >= c->n_layers || !scheme) return DC_ERR_ARG;
    const dc_layer_rt& L = c->L[layer];
    if (L.d.kind != DC_CONV || !c->executable) { *scheme = -1; return DC_OK; }
    if (!dc_conv_bf16_supported(c, layer)) { *scheme = 0; return DC_OK; }
    *scheme = (L.tc_mt > 0 ? L.tc_mt : 1) + (L.flat ? 7 : 0);
    return DC_OK;
}

int dc_cache_layer_regions(dc_cache* c, int layer, dc_region** regions_dev, int32_t** n_dev)
{
    if (!c || layer < -1 || layer >= c->n_layers || !regions_dev) return DC_ERR_ARG;
    *regions_dev = layer < 0 ? c->regions0 : c->table + (size_t)c->S * c->max_regions * layer;
    if (n_dev) *n_dev = c->n_regions;
    return DC_OK;
}

int dc_cache_counters(dc_cache* c, int64_t* reused_px_host, int64_t* frames_cached, int64_t* frames_full)
{
    if (!c) return DC_ERR_ARG;
    DC_CUDA(cudaStreamSynchronize(c->stream));
    if (reused_px_host)
        DC_CUDA(cudaMemcpy(reused_px_host, c->reused_total, sizeof(int64_t) * c->n_layers, cudaMemcpyDeviceToHost));
    if (frames_cached) *frames_cached = c->frames_cached;
    if (frames_full) *frames_full = c->frames_full;
    return DC_OK;
}

int dc_get_status(dc_cache* c, int32_t* status_host)
{
    if (!c || !status_host) return DC_ERR_ARG;
    DC_CUDA(cudaStreamSynchronize(c->stream));
    DC_CUDA(cudaMemcpy(status_host, c->status, sizeof(int32_t), cudaMemcpyDeviceToHost));
    return DC_OK;
}

const char* dc_strerror(int status)
{
    switch (status) {
    case DC_OK: return "ok";
    case DC_ERR_ARG: return "invalid argument";
    case DC_ERR_CONFIG: return "unsupported configuration";
    case DC_ERR_ALLOC: return "allocation failed";
    case DC_ERR_CUDA: return g_last_cuda_error[0] ? g_last_cuda_error : "CUDA call failed";
    case DC_ERR_OVERFLOW: return "more rectangles than max_regions";
    case DC_ERR_TIMEOUT: return "device-side wait timed out";
    case DC_ERR_STATE: return "call not valid in this state";
    case DC_ERR_LIMIT: return "size beyond a fixed built-in limit (dc_search_blocks_noalloc: at most 64 streams)";
    default: return "unknown status";
    }
}

}  // extern "C"
