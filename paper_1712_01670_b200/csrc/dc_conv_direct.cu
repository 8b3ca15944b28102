// Partial convolution on CUDA cores (Section 5, "Reuse", third step: convolve only the
// pixels that were not filled from the cache).
//
// Used for float32 networks, whose 1e-4 accuracy bound rules out tensor-core input formats,
// for layer shapes the tensor-core kernel does not take, and for grouped convolutions.  One CTA of 128 threads owns one
// dirty 16x8 output tile and a group of 32 output channels; thread t owns pixel t and keeps 32
// float accumulators.  Weights for one kernel row and 8 input channels are staged in shared
// memory as floats [kx][ci][co] and read as broadcast float4; inputs come straight from the
// NHWC map (8 consecutive channels per load).  The epilogue adds the bias, applies ReLU and
// writes only pixels whose bit in the tile's reuse bitmap is clear.
#include "dc_common.cuh"

namespace {

constexpr int CO_T = 32;     // output channels per CTA
constexpr int CI_T = 8;      // input channels per staging step
constexpr int MAX_KW = 11;

template <typename T> __device__ __forceinline__ float ld_f(const T* p);
template <> __device__ __forceinline__ float ld_f<float>(const float* p) { return __ldg(p); }
template <> __device__ __forceinline__ float ld_f<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ T st_f(float v);
template <> __device__ __forceinline__ float st_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 st_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

struct ConvArgs {
    const void* in; const void* w; const float* bias; void* out;
    const int32_t* tile_list; const int32_t* tile_count; const uint32_t* masks;
    int Hi, Wi, Ci, Ho, Wo, Co, kh, kw, sh, sw, ph, pw, relu, tiles_x, tiles_y;
    int Cig, Cog, co_blocks;     // grouped convolution: input / output channels per group, CTAs (of CO_T channels) per group
};

template <typename T>
__global__ void __launch_bounds__(DC_TILE_PX) k_conv_direct(ConvArgs a)
{
    __shared__ __align__(16) float wsm[MAX_KW * CI_T * CO_T];
    const T* in = (const T*)a.in; const T* wt = (const T*)a.w; T* out = (T*)a.out;
    const int tid = threadIdx.x, prow = tid / DC_TILE_W, pcol = tid % DC_TILE_W;
    // blockIdx.y = (group, block of CO_T output channels inside the group): a CTA never straddles two groups
    const int grp = blockIdx.y / a.co_blocks, co0 = grp * a.Cog + (blockIdx.y % a.co_blocks) * CO_T;
    const int con = min(CO_T, (grp + 1) * a.Cog - co0);
    const int ci_base = grp * a.Cig;                              // the group's first input channel
    const int per = a.tiles_x * a.tiles_y;
    const int n_tiles = *a.tile_count;
    for (int ti = blockIdx.x; ti < n_tiles; ti += gridDim.x) {
        const int tile = a.tile_list[ti];
        const int s = tile / per, t = tile - s * per, ty = t / a.tiles_x, tx = t - ty * a.tiles_x;
        const int oy = ty * DC_TILE_H + prow, ox = tx * DC_TILE_W + pcol;
        const bool in_map = oy < a.Ho && ox < a.Wo;
        const uint32_t mword = a.masks[(size_t)tile * 4 + (DC_TILE_BIT(prow, pcol) >> 5)];
        const bool reused = (mword >> (DC_TILE_BIT(prow, pcol) & 31)) & 1u;
        const bool active = in_map && !reused;
        float acc[CO_T];
#pragma unroll
        for (int i = 0; i < CO_T; ++i) acc[i] = 0.f;
        const T* in_s = in + (size_t)s * a.Hi * a.Wi * a.Ci;
        for (int ky = 0; ky < a.kh; ++ky) {
            const int iy = oy * a.sh - a.ph + ky;
            for (int ci0 = 0; ci0 < a.Cig; ci0 += CI_T) {
                const int cn = min(CI_T, a.Cig - ci0);
                __syncthreads();
                for (int e = tid; e < a.kw * CI_T * CO_T; e += DC_TILE_PX) {
                    int co = e % CO_T, ci = (e / CO_T) % CI_T, kx = e / (CO_T * CI_T);
                    float v = 0.f;
                    if (co < con && ci < cn)
                        v = ld_f(wt + (((size_t)(co0 + co) * a.kh + ky) * a.kw + kx) * a.Cig + ci0 + ci);
                    wsm[e] = v;
                }
                __syncthreads();
                if (!active || iy < 0 || iy >= a.Hi) continue;
                for (int kx = 0; kx < a.kw; ++kx) {
                    const int ix = ox * a.sw - a.pw + kx;
                    if (ix < 0 || ix >= a.Wi) continue;
                    const T* ap = in_s + ((size_t)iy * a.Wi + ix) * a.Ci + ci_base + ci0;
                    float av[CI_T];
#pragma unroll
                    for (int ci = 0; ci < CI_T; ++ci) av[ci] = ci < cn ? ld_f(ap + ci) : 0.f;
                    const float4* wp = (const float4*)(wsm + kx * CI_T * CO_T);
#pragma unroll
                    for (int ci = 0; ci < CI_T; ++ci) {
#pragma unroll
                        for (int q = 0; q < CO_T / 4; ++q) {
                            float4 w4 = wp[ci * (CO_T / 4) + q];
                            acc[4 * q + 0] = fmaf(av[ci], w4.x, acc[4 * q + 0]);
                            acc[4 * q + 1] = fmaf(av[ci], w4.y, acc[4 * q + 1]);
                            acc[4 * q + 2] = fmaf(av[ci], w4.z, acc[4 * q + 2]);
                            acc[4 * q + 3] = fmaf(av[ci], w4.w, acc[4 * q + 3]);
                        }
                    }
                }
            }
        }
        if (active) {
            T* op = out + (((size_t)s * a.Ho + oy) * a.Wo + ox) * a.Co + co0;
#pragma unroll
            for (int i = 0; i < CO_T; ++i) {
                if (i < con) {
                    float v = acc[i] + a.bias[co0 + i];
                    if (a.relu) v = fmaxf(v, 0.f);
                    op[i] = st_f<T>(v);
                }
            }
        }
    }
}

template <typename T>
__global__ void k_convert_weights(const float* src, size_t n, T* dst)
{
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        dst[i] = st_f<T>(src[i]);
}

}  // namespace

int dc_conv_bf16_supported(const dc_cache* c, int layer);
int dc_launch_conv_bf16(dc_cache* c, int layer, const void* in, void* out, const int32_t* tile_list,
                        const int32_t* tile_count, const uint32_t* masks, int max_tiles);

int dc_launch_conv(dc_cache* c, int layer, const void* in, void* out, const int32_t* tile_list,
                   const int32_t* tile_count, const uint32_t* masks, int max_tiles)
{
    dc_layer_rt& L = c->L[layer];
    if (L.s2d_s) {                                                // the rewritten layer reads the block map of its input
        dc_prof_scope ps(c, DC_ST_CONV);
        const int rc = dc_launch_s2d(c, layer, in);
        if (rc != DC_OK) return rc;
        in = L.in_s2d;
    }
    if (c->cfg.dtype == DC_BF16 && dc_conv_bf16_supported(c, layer))
        return dc_launch_conv_bf16(c, layer, in, out, tile_list, tile_count, masks, max_tiles);
    ConvArgs a;
    a.in = in; a.w = L.weight; a.bias = L.bias; a.out = out;
    a.tile_list = tile_list; a.tile_count = tile_count; a.masks = masks;
    a.Hi = L.in_h; a.Wi = L.in_w; a.Ci = L.d.cin; a.Ho = L.d.out_h; a.Wo = L.d.out_w; a.Co = L.d.cout;
    a.kh = L.d.kh; a.kw = L.d.kw; a.sh = L.d.sh; a.sw = L.d.sw; a.ph = L.d.ph; a.pw = L.d.pw; a.relu = L.d.relu;
    a.tiles_x = L.tiles_x; a.tiles_y = L.tiles_y;
    const int G = L.d.groups > 1 ? L.d.groups : 1;
    a.Cig = L.d.cin / G; a.Cog = L.d.cout / G; a.co_blocks = dc_div_up(a.Cog, CO_T);
    int co_groups = G * a.co_blocks;
    int gx = max_tiles < 1 ? 1 : max_tiles;
    int cap = dc_div_up(c->num_sms * 8, co_groups);
    if (gx > cap) gx = cap;
    dim3 grid(gx, co_groups);
    dc_prof_scope ps(c, DC_ST_CONV);
    if (c->cfg.dtype == DC_BF16) k_conv_direct<__nv_bfloat16><<<grid, DC_TILE_PX, 0, c->stream>>>(a);
    else k_conv_direct<float><<<grid, DC_TILE_PX, 0, c->stream>>>(a);
    c->launches += 1;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}

int dc_pack_weights_bf16(dc_cache* c, int layer);

int dc_pack_weights(dc_cache* c, int layer, const float* w_dev, const float* b_dev)
{
    dc_layer_rt& L = c->L[layer];
    size_t n = (size_t)L.d.cout * L.d.kh * L.d.kw * (L.d.cin / (L.d.groups > 1 ? L.d.groups : 1));
    if (L.d.kw > MAX_KW) return DC_ERR_CONFIG;
    DC_CUDA(cudaMalloc(&L.weight, n * c->elt));
    DC_CUDA(cudaMalloc((void**)&L.bias, sizeof(float) * L.d.cout));
    c->bytes += n * c->elt + sizeof(float) * L.d.cout;
    int grid = (int)((n + 255) / 256); if (grid > c->num_sms * 8) grid = c->num_sms * 8;
    if (c->cfg.dtype == DC_BF16) k_convert_weights<__nv_bfloat16><<<grid, 256, 0, c->stream>>>(w_dev, n, (__nv_bfloat16*)L.weight);
    else k_convert_weights<float><<<grid, 256, 0, c->stream>>>(w_dev, n, (float*)L.weight);
    DC_CUDA(cudaGetLastError());
    DC_CUDA(cudaMemcpyAsync(L.bias, b_dev, sizeof(float) * L.d.cout, cudaMemcpyDeviceToDevice, c->stream));
    if (c->cfg.dtype == DC_BF16) {
        if (dc_s2d_eligible(c, L.d)) {                            // from here on the layer is the stride-1 one
            const int rc = dc_s2d_rewrite(c, layer);
            if (rc != DC_OK) return rc;
        }
        return dc_pack_weights_bf16(c, layer);
    }
    return DC_OK;
}
