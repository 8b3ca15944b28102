// Internal declarations shared by the translation units of libdeepcache.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "deepcache.h"

#define DC_TILE_H 16         // output tile of the partial convolution: 16 rows x 8 columns
#define DC_TILE_W 8          // = 128 output pixels = the M dimension of one tensor-core tile; 8 columns = one
#define DC_TILE_PX (DC_TILE_H * DC_TILE_W)   // 8-row operand group per image row (see dc_conv_bf16.cu)
// Reuse bitmap of a tile: 128 bits, bit (row * DC_TILE_W + col), in four 32-bit words.
#define DC_TILE_BIT(row, col) ((row) * DC_TILE_W + (col))

#define DC_CUDA(call)                                            \
    do {                                                         \
        cudaError_t e__ = (call);                                \
        if (e__ != cudaSuccess) { dc_note_cuda_error(e__, __FILE__, __LINE__); return DC_ERR_CUDA; } \
    } while (0)

void dc_note_cuda_error(cudaError_t e, const char* file, int line);

// Stages timed by the optional event profiler (dc_cache_profile).
enum dc_stage { DC_ST_SEARCH = 0, DC_ST_VERIFY, DC_ST_MERGE, DC_ST_PROPAGATE, DC_ST_CLASSIFY_COPY, DC_ST_CONV,
                DC_ST_INPUT, DC_ST_POINTWISE, DC_ST_KEY_UPDATE, DC_ST_COUNT };

struct dc_prof;      // event pool, allocated when profiling is switched on

// A tensor map (CUtensorMap, 128 bytes) encoded for one base address and one operand scheme, kept so that a launch
// need not encode it again.  A layer's input alternates between at most two buffers (its producer's ping-pong maps).
struct dc_tm_slot {
    const void* base; int code, bn; bool valid;
    alignas(64) unsigned char map[128];
};

struct dc_layer_rt {
    dc_layer_desc d;
    int in_h, in_w;                 // size of the input map (or of the frame)
    int tiles_x, tiles_y;           // cached layers: 16 x 8 output tiles per stream
    // Flat tiles (convolutions on small or narrow maps): a tile is 16 consecutive GROUPS of 8 pixels of one image row,
    // groups numbered through rows, then streams: (stream * out_h + y) * gpr + column group.  A tile is then full
    // whatever the map's height, and across streams; only a row's last group can hold fewer than 8 pixels.
    int flat;                       // 1: this layer's tile list, bitmaps and convolution use flat tiles
    int gpr;                        // groups per image row = ceil(out_w / 8)
    int tiles_flat;                 // ceil(S * out_h * gpr / 16)
    void* map[2];                   // conv: current / cached output (ping-pong); others: map[0]
    int cur;                        // conv: which of map[] holds the newest output
    size_t map_bytes;               // bytes of one map, all streams
    void* weight;                   // conv: [cout][kh][kw][cin] in the cache dtype
    float* bias;                    // conv: [cout]
    void* weight_packed;            // conv, bf16: K-major tensor-core layout (see dc_conv_bf16.cu)
    int k_packed;                   // padded reduction length of weight_packed
    int tc_ctas;                    // conv, bf16: CTAs per SM the tuned launch uses (1 or 2)
    int tc_ew;                      // conv, bf16: epilogue warps per CTA (4, or 8 with one CTA per SM); 0 = 4
    int tc_mt, tc_bn;               // conv, bf16: tuned tiles per work item (3, 4: patch-reuse kernel with 1, 2; 5, 6: column-slab kernel) and
                                    // channels per block (0 = default)
    void* weight_halo;              // conv, bf16: weights packed for the patch-reuse and column-slab kernels
    int halo_bn;                    // channels per block that packing is grouped by
    void* in_padded;                // conv, bf16, cin <= 8: input with channels padded to 8
    void* in_s2d;                   // conv, bf16, strided over few channels: the space-to-depth copy of the input the rewritten layer reads (dc_conv_s2d.cu)
    int s2d_s, s2d_py, s2d_px, s2d_cin, s2d_hi, s2d_wi;   // ... its block size (0: layer as declared), leading zero rows / columns, and the input as declared
    uint32_t* masks;                // conv: [S][tiles_y][tiles_x][4] reuse bitmap of each tile
    int32_t* dirty_list;            // conv: compacted tiles needing computation
    int32_t* all_list;              // conv: every tile (used by full frames)
    dc_tm_slot tm_a[4], tm_b;       // conv, bf16: tensor maps of the input (two bases, two channel groups) and of the weights
    int tm_next;                    // which of tm_a[] a new input base replaces
};

// Everything one run of the matcher writes.  Two sets exist so that the matcher may already work on the
// next frame (dc_lookahead_frame) while inference of the current frame still reads its own set.
struct dc_match_set {
    int16_t* blk_mv; uint32_t* blk_sse; uint8_t* matched; uint16_t* run_end; int32_t* mv_acc; uint4* long_list;
    int32_t* gmv; dc_region* regions0; int32_t* n_regions;
};

struct dc_cache {
    dc_config cfg;
    int n_layers;
    dc_layer_rt L[DC_MAX_LAYERS];
    cudaStream_t stream;
    int S, Gx, Gy, max_regions;
    int elt;                        // bytes per map element
    bool executable;                // every layer kind has an execution kernel
    bool key_valid;
    int64_t frame_idx;
    int64_t launches;
    size_t bytes;

    uint8_t* key[3];                // key frames [S][H][key_pitch]: key[key_cur] is the cached previous frame,
    int key_cur;                    // key[(key_cur + 1) % 3] receives the frame being processed or looked ahead
    dc_match_set mset[2];           // the members blk_mv ... n_regions below alias mset[mset_cur]
    int mset_cur;
    cudaStream_t la_stream;         // dc_lookahead_frame: matcher of the next frame beside the current inference
    cudaEvent_t ev_key, ev_match;   // main stream: frame copied in; side stream: lookahead finished
    const uint8_t* la_frame; size_t la_pitch; bool la_matched;
    bool last_refreshed;
    bool overlap_mode;              // the last frame was looked ahead: the next one's matching will run beside this inference
    void* classify_table; int n_cached, classify_warps;   // all cached layers' classification in one launch (dc_regions.cu)
    size_t key_pitch;
    int num_sms;
    int device;                     // ordinal of the device the cache lives on
    int debug_stall_ms;             // > 0: the next tensor-core convolution launch is made to time out (tests)
    uint8_t* staging[2];            // device copies of host frames for dc_infer_frame_host (one in use, one prefetching)
    cudaStream_t copy_stream;       // dc_prefetch_frame_host copies on its own stream
    cudaEvent_t copied[2];
    const uint8_t* prefetched[2]; size_t prefetched_pitch[2];   // host frame whose copy each buffer holds, or NULL
    uint32_t sse_limit[4];          // PSNR test as an SSE bound, index = 2 * (bottom edge) + (right edge)

    int16_t* blk_mv;                // [S][Gy][Gx][2]
    uint32_t* blk_sse;              // [S][Gy][Gx]
    uint8_t* matched;               // [S][Gy][Gx]
    uint16_t* run_end;              // [S][Gy][Gx] Step 5: end column of the run starting at each block, else 0
    int32_t* mv_acc;                // [S][4]: sum dx, sum dy, K, n_matched; then 4 words of counters
    uint4* long_list;               // [S][Gy][Gx] diamond walks handed to the second search phase
    int32_t* gmv;                   // [S][3]: Mx, My, K
    dc_region* regions0;            // [S][max_regions] rectangles on the frame
    int32_t* n_regions;             // [S]
    dc_region* table;               // [n_layers][S][max_regions]
    dc_layer_desc* layers_dev;      // [n_layers]
    int32_t* in_hw_dev;             // [n_layers][2]
    int32_t* dirty_count;           // [n_layers]
    int32_t* all_count;             // [n_layers]
    int32_t* reuse_px;              // [n_layers][S]
    int32_t* alive;                 // [n_layers][S] rectangles not yet eroded away (directly behind reuse_px)
    uint32_t* zero_masks;           // all-zero reuse bitmap shared by full frames
    int32_t* status;                // device status word
    void* input_map;                // frame / 255 as a map, [S][H][W][3]
    void* pix_lut;                  // 256 entries: pixel value -> map element
    void* stats_pinned;             // host staging for statistics
    unsigned long long* reused_total; // [n_layers] reused output pixels summed over all frames so far
    int64_t frames_cached, frames_full;
    dc_prof* prof;
};

// Records a start / stop event pair around the enclosed launches when profiling is on.
struct dc_prof_scope {
    dc_cache* c; int stage;
    dc_prof_scope(dc_cache* cache, int st);
    ~dc_prof_scope();
};

static inline int dc_div_up(int a, int b) { return (a + b - 1) / b; }
// number of tiles of a cached layer in the tile geometry it uses
static inline int dc_layer_tiles(const dc_cache* c, const dc_layer_rt& L) { return L.flat ? L.tiles_flat : L.tiles_x * L.tiles_y * c->S; }
// device counter "all tiles" for full frames: [n_layers] for 16 x 8 tiles, then [n_layers] for flat tiles
static inline const int32_t* dc_all_count(const dc_cache* c, int layer) { return c->all_count + (c->L[layer].flat ? c->n_layers : 0) + layer; }

// A kernel's opt-in to more than 48 KB of dynamic shared memory (cudaFuncSetAttribute) holds for one device only.
// One of these per call site remembers on which devices it has been made.  Two threads may both find it unset and
// both set it: same value, harmless.
struct dc_once_per_device {
    bool done[64];
    bool first(int dev)
    {
        if (dev < 0 || dev >= 64) return true;        // beyond the table: set it every time
        if (done[dev]) return false;
        done[dev] = true;
        return true;
    }
};

// ---- kernels' host-side launchers (each returns DC_OK or DC_ERR_CUDA) ----
int dc_launch_copy_frame(dc_cache* c, const uint8_t* frame, size_t pitch, uint8_t* dst);
int dc_launch_match(dc_cache* c, const uint8_t* cur_key, const uint8_t* prev_key);   // both in key-frame layout
void dc_use_match_set(dc_cache* c, int k);
int dc_launch_propagate(dc_cache* c, const dc_region* in, const int32_t* n_in, int layer_end);
int dc_launch_classify_copy(dc_cache* c, int layer, const dc_region* regions, const int32_t* n_regions,
                            const void* prev_out, void* out);
int dc_launch_conv(dc_cache* c, int layer, const void* in, void* out, const int32_t* tile_list,
                   const int32_t* tile_count, const uint32_t* masks, int max_tiles);
int dc_launch_input_map(dc_cache* c, const uint8_t* frame, size_t pitch);
int dc_launch_resize(dc_cache* c, int layer, const uint8_t* frame, size_t pitch);   // frame: 16-byte aligned rows
int dc_launch_maxpool(dc_cache* c, int layer, const void* in, void* out, const uint32_t* masks);
int dc_launch_lrn(dc_cache* c, int layer, const void* in, void* out, const uint32_t* masks);
int dc_launch_concat(dc_cache* c, int layer, const void* a, int ca, const void* b, int cb);
int dc_launch_add(dc_cache* c, int layer, const void* a, const void* b);
int dc_launch_relu(dc_cache* c, int layer, const void* a);
int dc_pack_weights(dc_cache* c, int layer, const float* w_dev, const float* b_dev);
// true for layers that keep their last output as cached values: convolutions, and max pooling / LRN when cfg.cache_pool
bool dc_layer_cached(const dc_cache* c, int layer);
int dc_build_classify_table(dc_cache* c);
int dc_launch_classify_all(dc_cache* c, int cur);
int dc_conv_bf16_autotune(dc_cache* c, int layer, const void* in);
bool dc_s2d_eligible(const dc_cache* c, const dc_layer_desc& d);
int dc_s2d_rewrite(dc_cache* c, int layer);
int dc_launch_s2d(dc_cache* c, int layer, const void* in);
int dc_conv_bf16_supported(const dc_cache* c, int layer);    // 1 when the layer runs on the tensor-core kernels
