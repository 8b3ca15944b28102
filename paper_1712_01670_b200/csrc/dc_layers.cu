// Layers that are computed in full every frame (Section 5: only convolutions are cached):
// frame -> network input, area resize, max pooling, residual add, ReLU.  All are bandwidth
// bound: one pass over input and output.
#include "dc_common.cuh"

namespace {

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// round a double to bfloat16, nearest even, without passing through float
__device__ __forceinline__ __nv_bfloat16 double_to_bf16(double v)
{
    if (v == 0.0) return __float2bfloat16_rn(0.f);
    int e = ilogb(v);
    if (e < -126) e = -126;
    double q = ldexp(rint(ldexp(v, 7 - e)), e - 7);   // exactly representable in bfloat16
    return __float2bfloat16_rn((float)q);
}
template <typename T> __device__ __forceinline__ T from_d(double v);
template <> __device__ __forceinline__ float from_d<float>(double v) { return (float)v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_d<__nv_bfloat16>(double v) { return double_to_bf16(v); }

// pixel value -> map element through a 256-entry table (pixel / 255 in the map's type)
template <typename T>
__global__ void k_input_map(const uint8_t* frame, size_t pitch, int W, int H, int S, const T* lut, T* out)
{
    __shared__ T sl[256];
    if (threadIdx.x < 256) sl[threadIdx.x] = lut[threadIdx.x];
    __syncthreads();
    const int row_elems = W * 3;
    const size_t total = (size_t)S * H * row_elems;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        size_t row = i / row_elems; int x = (int)(i - row * row_elems);
        out[i] = sl[frame[row * pitch + x]];
    }
}

// Box average of the frame: output (oy, ox) is the mean over rows [floor(oy H / Ho),
// ceil((oy + 1) H / Ho) - 1] and the like columns, divided by 255.  One warp per output pixel;
// lanes stride over the source bytes of each span row (contiguous), integer sums.
template <typename T>
__global__ void __launch_bounds__(256) k_resize_area(const uint8_t* frame, size_t pitch, int W, int H, int S,
                                                     int Wo, int Ho, T* out)
{
    const int lane = threadIdx.x & 31;
    const long long wid = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (wid >= (long long)S * Ho * Wo) return;
    int ox = (int)(wid % Wo); long long t = wid / Wo; int oy = (int)(t % Ho); int s = (int)(t / Ho);
    int y0 = (int)((long long)oy * H / Ho), y1 = (int)(((long long)(oy + 1) * H + Ho - 1) / Ho) - 1;
    int x0 = (int)((long long)ox * W / Wo), x1 = (int)(((long long)(ox + 1) * W + Wo - 1) / Wo) - 1;
    const uint8_t* base = frame + ((size_t)s * H + y0) * pitch + (size_t)x0 * 3;
    const int nb = (x1 - x0 + 1) * 3, rows = y1 - y0 + 1;
    uint32_t c0 = 0, c1 = 0, c2 = 0;
    for (int i = lane; i < nb * rows; i += 32) {
        int r = i / nb, b = i - r * nb;
        uint32_t v = base[(size_t)r * pitch + b];
        int ch = b % 3;
        c0 += ch == 0 ? v : 0; c1 += ch == 1 ? v : 0; c2 += ch == 2 ? v : 0;
    }
    c0 = __reduce_add_sync(0xffffffffu, c0); c1 = __reduce_add_sync(0xffffffffu, c1);
    c2 = __reduce_add_sync(0xffffffffu, c2);
    if (lane < 3) {
        uint32_t sum = lane == 0 ? c0 : (lane == 1 ? c1 : c2);
        double mean = (double)sum / ((double)(rows * (x1 - x0 + 1)) * 255.0);
        out[(size_t)wid * 3 + lane] = from_d<T>(mean);
    }
}

template <typename T>
__global__ void k_maxpool(const T* in, int Hi, int Wi, int C, int S, dc_layer_desc L, T* out)
{
    const size_t total = (size_t)S * L.out_h * L.out_w * C;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        int c = (int)(i % C); size_t t = i / C;
        int ox = (int)(t % L.out_w); t /= L.out_w;
        int oy = (int)(t % L.out_h); int s = (int)(t / L.out_h);
        float m = -INFINITY;
        for (int ky = 0; ky < L.kh; ++ky) {
            int iy = oy * L.sh - L.ph + ky;
            if (iy < 0 || iy >= Hi) continue;
            for (int kx = 0; kx < L.kw; ++kx) {
                int ix = ox * L.sw - L.pw + kx;
                if (ix < 0 || ix >= Wi) continue;
                m = fmaxf(m, to_f(in[(((size_t)s * Hi + iy) * Wi + ix) * C + c]));
            }
        }
        out[i] = from_f<T>(m);
    }
}

template <typename T>
__global__ void k_add(const T* a, const T* b, size_t n, int relu, T* out)
{
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        float v = to_f(a[i]) + to_f(b[i]);
        if (relu) v = fmaxf(v, 0.f);
        out[i] = from_f<T>(v);
    }
}

template <typename T>
__global__ void k_relu(const T* a, size_t n, T* out)
{
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        out[i] = from_f<T>(fmaxf(to_f(a[i]), 0.f));
}

inline int grid_for(size_t n, int block) { size_t g = (n + block - 1) / block; return (int)(g > 148 * 16 ? 148 * 16 : (g ? g : 1)); }

}  // namespace

#define DISPATCH(c, expr_f32, expr_bf16) do { if ((c)->cfg.dtype == DC_BF16) { expr_bf16; } else { expr_f32; } } while (0)

int dc_launch_input_map(dc_cache* c, const uint8_t* frame, size_t pitch)
{
    size_t n = (size_t)c->S * c->cfg.height * c->cfg.width * 3;
    int W = c->cfg.width, H = c->cfg.height;
    dc_prof_scope ps(c, DC_ST_INPUT);
    DISPATCH(c,
        (k_input_map<float><<<grid_for(n, 256), 256, 0, c->stream>>>(frame, pitch, W, H, c->S, (const float*)c->pix_lut, (float*)c->input_map)),
        (k_input_map<__nv_bfloat16><<<grid_for(n, 256), 256, 0, c->stream>>>(frame, pitch, W, H, c->S, (const __nv_bfloat16*)c->pix_lut, (__nv_bfloat16*)c->input_map)));
    c->launches += 1;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}

int dc_launch_resize(dc_cache* c, int layer, const uint8_t* frame, size_t pitch)
{
    dc_layer_rt& L = c->L[layer];
    long long warps = (long long)c->S * L.d.out_h * L.d.out_w;
    int grid = (int)((warps + 7) / 8);
    dc_prof_scope ps(c, DC_ST_INPUT);
    DISPATCH(c,
        (k_resize_area<float><<<grid, 256, 0, c->stream>>>(frame, pitch, c->cfg.width, c->cfg.height, c->S, L.d.out_w, L.d.out_h, (float*)L.map[0])),
        (k_resize_area<__nv_bfloat16><<<grid, 256, 0, c->stream>>>(frame, pitch, c->cfg.width, c->cfg.height, c->S, L.d.out_w, L.d.out_h, (__nv_bfloat16*)L.map[0])));
    c->launches += 1;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}

int dc_launch_maxpool(dc_cache* c, int layer, const void* in)
{
    dc_layer_rt& L = c->L[layer];
    size_t n = (size_t)c->S * L.d.out_h * L.d.out_w * L.d.cout;
    dc_prof_scope ps(c, DC_ST_POINTWISE);
    DISPATCH(c,
        (k_maxpool<float><<<grid_for(n, 256), 256, 0, c->stream>>>((const float*)in, L.in_h, L.in_w, L.d.cout, c->S, L.d, (float*)L.map[0])),
        (k_maxpool<__nv_bfloat16><<<grid_for(n, 256), 256, 0, c->stream>>>((const __nv_bfloat16*)in, L.in_h, L.in_w, L.d.cout, c->S, L.d, (__nv_bfloat16*)L.map[0])));
    c->launches += 1;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}

int dc_launch_add(dc_cache* c, int layer, const void* a, const void* b)
{
    dc_layer_rt& L = c->L[layer];
    size_t n = (size_t)c->S * L.d.out_h * L.d.out_w * L.d.cout;
    dc_prof_scope ps(c, DC_ST_POINTWISE);
    DISPATCH(c,
        (k_add<float><<<grid_for(n, 256), 256, 0, c->stream>>>((const float*)a, (const float*)b, n, L.d.relu, (float*)L.map[0])),
        (k_add<__nv_bfloat16><<<grid_for(n, 256), 256, 0, c->stream>>>((const __nv_bfloat16*)a, (const __nv_bfloat16*)b, n, L.d.relu, (__nv_bfloat16*)L.map[0])));
    c->launches += 1;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}

int dc_launch_relu(dc_cache* c, int layer, const void* a)
{
    dc_layer_rt& L = c->L[layer];
    size_t n = (size_t)c->S * L.d.out_h * L.d.out_w * L.d.cout;
    dc_prof_scope ps(c, DC_ST_POINTWISE);
    DISPATCH(c,
        (k_relu<float><<<grid_for(n, 256), 256, 0, c->stream>>>((const float*)a, n, (float*)L.map[0])),
        (k_relu<__nv_bfloat16><<<grid_for(n, 256), 256, 0, c->stream>>>((const __nv_bfloat16*)a, n, (__nv_bfloat16*)L.map[0])));
    c->launches += 1;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}
