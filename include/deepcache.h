/*
 * deepcache.h -- C ABI of the DeepCache hot path for NVIDIA B200 (sm_100a).
 *
 * DeepCache (arXiv 1712.01670) speeds up CNN inference on video by reusing,
 * per convolution layer, the previous frame's outputs wherever the new frame
 * matches the previous one.  This library implements the per-frame path:
 *
 *   Section 4  image block matching     dc_match_blocks
 *   Section 5  region propagation       dc_propagate_regions   (Table 2)
 *   Section 5  reuse inside convolution dc_conv_partial        (c_forward of Section 6)
 *   Sections 3, 5  the whole frame      dc_infer_frame         (with cache expiry)
 *
 * General rules
 *   - Every function returns DC_OK (0) or a negative dc_status; nothing throws
 *     or aborts across this boundary.  dc_strerror names a status.
 *   - "_dev" pointers are CUDA device memory owned by the caller; they must stay
 *     valid until the cache's stream has passed the call.  "_host" pointers are
 *     ordinary host memory.
 *   - All work is enqueued on the CUDA stream given to dc_cache_create and is
 *     asynchronous unless stated otherwise.
 *   - Environment switches read by the library (diagnostics only): DC_VERBOSE prints CUDA error strings and the
 *     per-layer kernel choices made by dc_cache_create; DC_CONV_NO_TUNE skips the per-layer timing and keeps the
 *     default work split; DC_NO_TENSOR_CORES runs every convolution on the CUDA-core kernel; DC_CONV_SCHEME=<1..6>
 *     restricts that timing to one operand scheme of the tensor-core convolution (used by the tests to reach each one).
 *   - Frames are uint8, interleaved HWC with 3 channels; n_streams frames are
 *     stacked, stream s starting at frame + s * height * pitch_bytes.
 *   - Feature maps are NHWC, N = n_streams, element type float (DC_FP32) or
 *     bfloat16 (DC_BF16).  Weights are given as float32 [cout][kh][kw][cin] and
 *     are converted by the library; biases stay float32.
 *   - A motion vector (dx, dy) points from a block of the current frame to its
 *     match in the previous frame: previous = current + (dx, dy)
 *     (Section 4, Step 2: (x'_i - x_i, y'_i - y_i)).
 *   - Region lists are slot-preserving: slot i of every layer descends from
 *     matcher rectangle i; a region that has eroded away is all zeros.
 */
#ifndef DEEPCACHE_H
#define DEEPCACHE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DC_MAX_LAYERS 128

typedef enum {
    DC_OK = 0,
    DC_ERR_ARG = -1,       /* null or inconsistent argument */
    DC_ERR_CONFIG = -2,    /* unsupported configuration or layer table */
    DC_ERR_ALLOC = -3,     /* device or host allocation failed */
    DC_ERR_CUDA = -4,      /* a CUDA call failed */
    DC_ERR_OVERFLOW = -5,  /* more rectangles than max_regions (device status word) */
    DC_ERR_TIMEOUT = -6,   /* a bounded device-side wait ran out (device status word) */
    DC_ERR_STATE = -7,     /* call not valid now (e.g. no cached frame yet) */
    DC_ERR_LIMIT = -8      /* size beyond a fixed built-in limit (dc_search_blocks_noalloc) */
} dc_status;

/* A reusable rectangle (Section 3: "(x, y, w, h) -> (x', y', w, h)").
 * (x, y, w, h): rectangle in the current frame or map; (sx, sy): origin of the
 * same-sized rectangle in the previous frame or cached map. */
typedef struct { int32_t x, y, w, h, sx, sy; } dc_region;

typedef enum {
    DC_CONV = 0, DC_MAXPOOL = 1, DC_RELU = 2, DC_ADD = 3, DC_CONCAT = 4,
    DC_RESIZE_AREA = 5, DC_LRN = 6, DC_FC = 7
} dc_layer_kind;

/* One layer.  in0 / in1: index of the producing layer, -1 = the input frame
 * (in1 is used by DC_ADD / DC_CONCAT only).  out_h, out_w: output size.
 * DC_CONV: kh x kw kernel, stride, padding, cin -> cout, optional fused ReLU, optionally in channel groups.
 * DC_MAXPOOL: floor mode, padded taps ignored.  DC_ADD: element-wise, optional ReLU.
 * DC_RESIZE_AREA: box average of the input frame (in0 must be -1) to out_h x out_w.
 * DC_LRN: local response normalisation inside each channel over a (2 ph + 1)^2 spatial window (the form Table 2's
 *   radius describes): b = a / (k + alpha / n^2 * sum of a^2 over the window)^beta, outside pixels count as zero;
 *   alpha, beta, k come from dc_config.  Executable when kh = kw = 2 ph + 1 and pw = ph.
 * DC_CONCAT: channels of in0 followed by those of in1.
 * DC_FC: fully connected; executable when kh, kw equal the input map's height and width (then it is the convolution
 *   whose kernel covers the whole map: weights [cout][kh][kw][cin], out 1 x 1, optional ReLU).  Table 2: nothing of
 *   its output is reusable.
 * A layer table with an LRN or FC layer of another shape is accepted for region propagation, but such a cache
 * cannot run dc_infer_frame.
 * Limit: an executable cache takes DC_CONV and DC_FC kernels of at most 11 columns (kw <= 11; any kh);
 * dc_cache_create returns DC_ERR_CONFIG for a wider one. */
typedef struct {
    int32_t kind, kh, kw, sh, sw, ph, pw, cin, cout, relu, in0, in1, out_h, out_w;
    int32_t groups;   /* DC_CONV only: grouped convolution (the cited AlexNet's form); 0 or 1 = ordinary.  Output channel
                         co belongs to group co / (cout / groups) and sees input channels group * cin / groups ...; both
                         cin and cout must be multiples of groups; weights [cout][kh][kw][cin / groups].  Must be 0 or 1
                         for every other kind. */
} dc_layer_desc;

/* The search unit of Step 2.  Exhaustive: every displacement within +-range.  Diamond: the paper's default
 * (Section 4).  Three step: the alternative Section 7.5 compares; nine-point passes with step S0, S0/2, ..., 1
 * where S0 is the largest power of two with 2 S0 - 1 <= range. */
typedef enum { DC_SEARCH_EXHAUSTIVE = 0, DC_SEARCH_DIAMOND = 1, DC_SEARCH_THREE_STEP = 2 } dc_search_kind;
typedef enum { DC_FP32 = 0, DC_BF16 = 1 } dc_dtype;
/* How matched blocks become rectangles.  DC_REGIONS_GLOBAL is the paper's Steps 3-5: one mean vector M per frame,
 * blocks verified at M, every rectangle displaced by M.  DC_REGIONS_PER_BLOCK is an extension with no counterpart
 * in the paper (Section 4 names the limit it lifts: content that moves against the global vector is lost):
 * a searched block is accepted with its own Step 2 vector when that match passes the threshold, and only
 * neighbours with the same vector merge, so each rectangle carries its own displacement.  The global vector
 * is still computed and reported.  Blocks skipped by skip_k have no vector and stay unmatched in this mode. */
typedef enum { DC_REGIONS_GLOBAL = 0, DC_REGIONS_PER_BLOCK = 1 } dc_region_mode;

/* The developer-facing knobs of Section 6 (threshold, block size, expiry) plus shapes. */
typedef struct {
    int32_t width, height, channels;   /* frame size in pixels; channels must be 3 */
    int32_t n_streams;                 /* independent video streams processed per call */
    int32_t block;                     /* block edge in pixels (Section 3 default 10), 4..32 */
    int32_t range;                     /* search range R: |dx|, |dy| <= R, 0..64 */
    int32_t search;                    /* dc_search_kind */
    int32_t skip_k;                    /* Step 2 searches only blocks on every skip_k-th row and column (Section 4,
                                          "k-skip"); 1 = every block; 1..16 */
    int32_t expire_n;                  /* full fresh frame every expire_n frames (default 10) */
    double  psnr_db;                   /* similarity threshold T in dB (default 20) */
    int32_t dtype;                     /* dc_dtype of maps and arithmetic inputs */
    int32_t max_regions;               /* rectangles per stream; 0 = worst case of the grid */
    int32_t region_mode;               /* dc_region_mode; 0 = the paper's global vector */
    int32_t cache_pool;                /* 1: max-pooling and LRN layers keep their last output and reuse it like convolutions
                                          (the extension Section 5 mentions; costs a second pooled map per layer).
                                          Applies to such layers whose pixel is a multiple of 16 bytes.  0 = the
                                          paper's choice: only convolutions are cached */
    double  lrn_alpha, lrn_beta, lrn_k;/* parameters of every DC_LRN layer; all three 0 selects 1e-4, 0.75, 1 */
} dc_config;

/* Per-stream outcome of one dc_infer_frame. */
typedef struct {
    int32_t refreshed;                 /* 1: full fresh frame (expiry or empty cache) */
    int32_t n_blocks, k_passed;        /* grid size; blocks whose best match passed (Step 3's K) */
    int32_t mvx, mvy;                  /* global motion (Mx, My) */
    int32_t n_matched, n_regions;      /* Step 4 matches; Step 5 rectangles */
    float   reuse_ratio[DC_MAX_LAYERS];/* per layer: reused / all output pixels (conv layers) */
} dc_frame_stats;

typedef struct dc_cache dc_cache;      /* opaque, owned by the library */

/* Builds a cache for one network and one frame geometry: validates, allocates the
 * key-frame buffer, two maps per convolution (current / cached), one per other layer,
 * region tables and tile lists, and converts the weights.  weights_dev[i] / bias_dev[i]
 * are float32 device arrays for DC_CONV layers and ignored (may be NULL) otherwise; they
 * are read during this call only.  cuda_stream is a cudaStream_t (NULL = default stream).
 * Synchronous.  Errors: DC_ERR_ARG, DC_ERR_CONFIG, DC_ERR_ALLOC, DC_ERR_CUDA. */
int dc_cache_create(const dc_config* cfg, const dc_layer_desc* layers, int n_layers,
                    const void* const* weights_dev, const void* const* bias_dev,
                    void* cuda_stream, dc_cache** out);

/* Frees everything the cache owns.  Synchronous. */
int dc_cache_destroy(dc_cache* cache);

/* Empties the cache: the next dc_infer_frame is a full fresh frame (Section 5, expiry). */
int dc_cache_reset(dc_cache* cache);

/* Device bytes held by the cache (cf. the memory overhead of Section 7.7). */
int dc_cache_bytes(const dc_cache* cache, size_t* bytes);

/* Stores frame_dev as the cached previous frame (the cache key of Section 3) without
 * running the network.  Lets dc_match_blocks be used on its own. */
int dc_cache_set_key(dc_cache* cache, const uint8_t* frame_dev, size_t pitch_bytes);

/* Section 4, Steps 1-5, current frame against the cached previous frame.
 *   block_mv_dev   int16  [S][Gy][Gx][2]  best (dx, dy) per block (Step 2)
 *   block_sse_dev  uint32 [S][Gy][Gx]     its sum of squared differences over 3 channels
 *                                         (blocks skipped by skip_k: vector (0, 0), SSE 0xFFFFFFFF)
 *   matched_dev    uint8  [S][Gy][Gx]     1 = properly matched at the global motion (Step 4)
 *   global_mv_dev  int32  [S][3]          Mx, My, K (Step 3)
 *   regions_dev    dc_region [S][max_regions], n_regions_dev int32 [S]   (Step 5)
 * Gx = ceil(width / block), Gy = ceil(height / block); edge blocks are clipped.
 * Any output pointer may be NULL (skipped).  Does not change the cache.
 * Errors: DC_ERR_ARG, DC_ERR_STATE (no cached frame), DC_ERR_CUDA. */
int dc_match_blocks(dc_cache* cache, const uint8_t* frame_dev, size_t pitch_bytes,
                    int16_t* block_mv_dev, uint32_t* block_sse_dev, uint8_t* matched_dev,
                    int32_t* global_mv_dev, dc_region* regions_dev, int32_t* n_regions_dev);

/* Section 5 "Propagation" (Table 2): carries frame-level rectangles through layers
 * 0 .. layer_end-1 and returns those of layers layer_begin .. layer_end-1.
 *   in_dev   dc_region [S][max_regions], n_in_dev int32 [S]: rectangles on the input frame
 *   out_dev  dc_region [layer_end-layer_begin][S][max_regions]
 *   n_out_dev int32 [layer_end-layer_begin][S] (slot count, equal to n_in; may be NULL)
 * Slots at or beyond max_regions are never written, whatever n_in_dev says.
 * Errors: DC_ERR_ARG, DC_ERR_CUDA. */
int dc_propagate_regions(dc_cache* cache, const dc_region* in_dev, const int32_t* n_in_dev,
                         int layer_begin, int layer_end, dc_region* out_dev, int32_t* n_out_dev);

/* Section 5 "Reuse" for convolution layer `layer` (c_forward(top, bottom, c_blob, c_regions)
 * of Section 6): output pixels inside a rectangle are copied from prev_out_dev at the mapped
 * position, all others are convolved (+bias, +ReLU) from in_map_dev.
 *   in_map_dev    [S][Hi][Wi][cin]   complete input map (bottom blob)
 *   prev_out_dev  [S][Ho][Wo][cout]  this layer's output for the previous frame (c_blob)
 *   regions_dev   dc_region [S][max_regions], n_regions_dev int32 [S]: rectangles in output
 *                 coordinates (c_regions); both NULL = plain full convolution
 *   out_map_dev   [S][Ho][Wo][cout]  (top blob); must not alias prev_out_dev
 * A count above max_regions is cut to max_regions.  A rectangle that does not lie inside the Ho x Wo map on
 * both sides (current and cached) is not reused -- its pixels are convolved like any other -- and the device
 * status word is set to DC_ERR_ARG (dc_get_status); no map is ever addressed outside its bounds.
 * Errors: DC_ERR_ARG, DC_ERR_CONFIG (not a convolution), DC_ERR_CUDA. */
int dc_conv_partial(dc_cache* cache, int layer, const void* in_map_dev, const void* prev_out_dev,
                    const dc_region* regions_dev, const int32_t* n_regions_dev, void* out_map_dev);

/* One frame per stream through the whole path: expiry check, matching, propagation,
 * every layer (convolutions partially, the rest in full), then the frame becomes the new
 * key and the convolution outputs the new cached values (Sections 3 and 5).
 *   out_map_dev     last layer's map, [S][Ho][Wo][cout]; may be NULL
 *   stats_host      dc_frame_stats [S] or NULL.  Non-NULL makes the call synchronous.
 * Errors: DC_ERR_ARG, DC_ERR_STATE (layer table not executable), DC_ERR_CUDA. */
int dc_infer_frame(dc_cache* cache, const uint8_t* frame_dev, size_t pitch_bytes,
                   void* out_map_dev, dc_frame_stats* stats_host);

/* Announces the frame that the NEXT dc_infer_frame will get, so that its matching (Steps 1-5) runs on a
 * side stream while the convolutions of the current frame are still running: Section 7.6 points out that
 * matching one image and inferring another can proceed at the same time.  Call it after dc_infer_frame
 * for frame t, with frame t+1; the next dc_infer_frame must then be given the same frame_dev and
 * pitch_bytes (any other frame simply discards the lookahead).  frame_dev must stay unchanged until that
 * call.  Results are identical with and without it.  The side stream has the lowest priority; when the
 * stream given to dc_cache_create has a higher one, the convolution kernels get the SMs first and the
 * matcher fills what they leave, which shortens the overlapped step further.
 * Errors: DC_ERR_ARG, DC_ERR_STATE (no frame inferred yet, or layer table not executable), DC_ERR_CUDA. */
int dc_lookahead_frame(dc_cache* cache, const uint8_t* frame_dev, size_t pitch_bytes);

/* Same as dc_infer_frame with HOST buffers: copies the frames to the device, runs the
 * path, copies the last map back, and waits.  frame_host should be pinned memory for
 * full copy speed.  out_map_host may be NULL. */
int dc_infer_frame_host(dc_cache* cache, const uint8_t* frame_host, size_t pitch_bytes,
                        void* out_map_host, dc_frame_stats* stats_host);

/* Starts the host-to-device copy of the NEXT frame on a separate stream, so it overlaps the frame being
 * computed (Section 7.6 notes that matching one image and inferring another can run at the same time).
 * A later dc_infer_frame_host with the same frame_host and pitch_bytes uses that copy instead of copying
 * again, and matches the prefetched frame on a side stream while the current one is computed (as
 * dc_lookahead_frame does).  Typical loop: prefetch(frame t+1), infer(frame t), prefetch(frame t+2), infer(frame t+1), ...
 * At most two frames can be pending (DC_ERR_STATE otherwise).  frame_host must stay unchanged until that call and should be
 * pinned memory (a pageable buffer makes the copy synchronous).  Errors: DC_ERR_ARG, DC_ERR_ALLOC, DC_ERR_CUDA. */
int dc_prefetch_frame_host(dc_cache* cache, const uint8_t* frame_host, size_t pitch_bytes);

/* Device address and size of the library-owned map of `layer` as of the last
 * dc_infer_frame (for inspection; valid until the next call on this cache). */
int dc_cache_layer_map(dc_cache* cache, int layer, void** map_dev, size_t* bytes);

/* Device address of the rectangles dc_infer_frame / dc_propagate_regions last computed for
 * `layer` ([S][max_regions]) and of their per-stream count ([S]). */
int dc_cache_layer_regions(dc_cache* cache, int layer, dc_region** regions_dev, int32_t** n_dev);

/* Which kernel family runs convolution layer `layer` (chosen at creation): -1 not an executable convolution,
 * 0 the CUDA-core kernel (fp32 caches, channel counts the tensor-core kernels cannot take), 1-9 a tensor-core
 * operand scheme (1, 2 tap by tap; 3, 4 input patch; 5, 6 column slabs; 7 column slabs on CTA pairs; 8, 9 tap by
 * tap on tiles made of 16 row pieces of 8 pixels taken across rows and streams, for small maps; grouped layers
 * run their scheme once per group).  For inspection and tests.  Errors: DC_ERR_ARG. */
int dc_cache_layer_conv_scheme(const dc_cache* cache, int layer, int32_t* scheme);

/* Waits for the stream and returns the device status word: DC_OK, or what a kernel recorded since the
 * last reset: DC_ERR_OVERFLOW (Step 5 found more rectangles than max_regions), DC_ERR_TIMEOUT (a bounded
 * device-side wait or walk ran out; the affected results are not valid), DC_ERR_ARG (a caller's rectangle
 * outside its map was ignored).  Synchronous. */
int dc_get_status(dc_cache* cache, int32_t* status_host);

/* Kernels of this library launched on this cache since creation (for reporting). */
int dc_cache_launches(const dc_cache* cache, int64_t* launches);

/* Optional per-stage timing with CUDA events on the cache's stream.  While enabled, every
 * kernel launch of the library is bracketed by an event pair.  dc_cache_profile waits for the
 * stream, adds up the pairs recorded since the last call and clears them.
 *   ms_host / launches_host: DC_PROFILE_STAGES entries each, indexed by dc_profile_stage. */
typedef enum {
    DC_PROF_SEARCH = 0, DC_PROF_VERIFY = 1, DC_PROF_MERGE = 2, DC_PROF_PROPAGATE = 3,
    DC_PROF_CLASSIFY_COPY = 4, DC_PROF_CONV = 5, DC_PROF_INPUT = 6, DC_PROF_POINTWISE = 7,
    DC_PROF_KEY_UPDATE = 8
} dc_profile_stage;
#define DC_PROFILE_STAGES 9
int dc_cache_set_profiling(dc_cache* cache, int enable);
int dc_cache_profile(dc_cache* cache, float* ms_host, int64_t* launches_host);

/* Running totals since creation or the last dc_cache_reset: reused output pixels per layer
 * (reused_px_host: n_layers entries, summed over streams and frames), frames served from the
 * cache and full fresh frames (each counts one call, not one stream).  Synchronous. */
int dc_cache_counters(dc_cache* cache, int64_t* reused_px_host, int64_t* frames_cached, int64_t* frames_full);

/* Block search without any allocation.  (The paper has no counterpart: this entry point exists
 * for callers that must not allocate device memory, so cannot create a dc_cache -- code running
 * where cudaMalloc is not allowed or not affordable, such as a processing loop whose memory was
 * fixed at start-up, or a plug-in whose host forbids allocation after initialisation.)
 *
 * Runs Steps 2 and 3 of the matcher on caller-owned frames: for each block of frame_dev the best
 * motion vector into prev_dev and its SSE, and per stream the rounded mean vector of the blocks
 * that pass the PSNR test.  Same definitions, candidate order and outputs as dc_match_blocks.
 * search must be DC_SEARCH_EXHAUSTIVE or DC_SEARCH_DIAMOND (three step search: DC_ERR_CONFIG).
 *   frame_dev, prev_dev   uint8 HWC frames, n_streams stacked, any alignment, row pitch pitch_bytes
 *   block_mv_dev   int16  [S][Gy][Gx][2],  block_sse_dev uint32 [S][Gy][Gx],  global_mv_dev int32 [S][3]
 *   cuda_stream    cudaStream_t the work is enqueued on (asynchronous)
 * Its only scratch memory is a fixed array inside the library (DC_NOALLOC_MAX_STREAMS x 16 bytes
 * = 1 KiB per GPU, held from library load to process exit).  The call never calls cudaMalloc,
 * cudaFree or any allocating routine.  All calls on one GPU share that array: each call clears what
 * it uses first, so calls must not overlap on the GPU (run them on one stream, or order them with
 * events); overlapping calls race and return wrong mean vectors.  The first call on a device looks
 * up the array's device address (cudaGetSymbolAddress); make that first call outside any stream
 * capture.
 * Errors: DC_ERR_ARG, DC_ERR_CONFIG (block, range, search, threshold out of range),
 * DC_ERR_LIMIT (n_streams > DC_NOALLOC_MAX_STREAMS, or device ordinal >= 64), DC_ERR_CUDA. */
#define DC_NOALLOC_MAX_STREAMS 64
int dc_search_blocks_noalloc(const uint8_t* frame_dev, const uint8_t* prev_dev, size_t pitch_bytes,
                             int32_t width, int32_t height, int32_t n_streams, int32_t block, int32_t range,
                             int32_t search, double psnr_db, int16_t* block_mv_dev, uint32_t* block_sse_dev,
                             int32_t* global_mv_dev, void* cuda_stream);

const char* dc_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* DEEPCACHE_H */
