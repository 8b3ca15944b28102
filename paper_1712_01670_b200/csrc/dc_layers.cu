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
// ceil((oy + 1) H / Ho) - 1] and the like columns, divided by 255.  One CTA per output row:
// pass 1 sums the span's source rows column-wise with coalesced 16-byte loads (row starts are
// 16-byte aligned in the library's frame copy) into shared memory; pass 2 sums each output's
// column span.  All sums are integers; the one division is done in double.
template <typename T>
__global__ void __launch_bounds__(256) k_resize_area(const uint8_t* frame, size_t pitch, int W, int H, int S,
                                                     int Wo, int Ho, T* out)
{
    extern __shared__ uint16_t colsum[];                       // [ceil16(W * 3)]
    const int oy = blockIdx.x % Ho, s = blockIdx.x / Ho;
    const int y0 = (int)((long long)oy * H / Ho), y1 = (int)(((long long)(oy + 1) * H + Ho - 1) / Ho) - 1;
    const int row_bytes = W * 3, chunks = (row_bytes + 15) >> 4;
    const uint8_t* base = frame + ((size_t)s * H + y0) * pitch;
    for (int c = threadIdx.x; c < chunks; c += blockDim.x) {
        uint32_t acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};            // 16 byte columns as 8 pairs of 16-bit sums
        for (int y = 0; y <= y1 - y0; ++y) {
            const uint4 v = __ldg((const uint4*)(base + (size_t)y * pitch + c * 16));
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                acc[2 * k] += __byte_perm(w[k], 0, 0x4140);    // bytes 0, 1 -> two 16-bit lanes
                acc[2 * k + 1] += __byte_perm(w[k], 0, 0x4342);
            }
        }
        uint4* dst = (uint4*)(colsum + c * 16);
        dst[0] = make_uint4(acc[0], acc[1], acc[2], acc[3]);
        dst[1] = make_uint4(acc[4], acc[5], acc[6], acc[7]);
    }
    __syncthreads();
    const int rows = y1 - y0 + 1;
    for (int t = threadIdx.x; t < Wo * 3; t += blockDim.x) {
        const int ox = t / 3, ch = t - ox * 3;
        const int x0 = (int)((long long)ox * W / Wo), x1 = (int)(((long long)(ox + 1) * W + Wo - 1) / Wo) - 1;
        uint32_t sum = 0;
        for (int x = x0; x <= x1; ++x) sum += colsum[x * 3 + ch];
        const double mean = (double)sum / ((double)(rows * (x1 - x0 + 1)) * 255.0);
        out[(((size_t)s * Ho + oy) * Wo + ox) * 3 + ch] = from_d<T>(mean);
    }
}

// 8 (bf16) or 4 (float) channels per thread with 16-byte loads; C must be a multiple of that.
template <typename T> struct Vec16;
template <> struct Vec16<float> {
    static constexpr int N = 4;
    static __device__ __forceinline__ uint4 vmax(uint4 a, uint4 b)
    {
        return make_uint4(__float_as_uint(fmaxf(__uint_as_float(a.x), __uint_as_float(b.x))),
                          __float_as_uint(fmaxf(__uint_as_float(a.y), __uint_as_float(b.y))),
                          __float_as_uint(fmaxf(__uint_as_float(a.z), __uint_as_float(b.z))),
                          __float_as_uint(fmaxf(__uint_as_float(a.w), __uint_as_float(b.w))));
    }
};
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int N = 8;
    static __device__ __forceinline__ uint32_t m2(uint32_t a, uint32_t b)
    {
        __nv_bfloat162 r = __hmax2(*reinterpret_cast<__nv_bfloat162*>(&a), *reinterpret_cast<__nv_bfloat162*>(&b));
        return *reinterpret_cast<uint32_t*>(&r);
    }
    static __device__ __forceinline__ uint4 vmax(uint4 a, uint4 b) { return make_uint4(m2(a.x, b.x), m2(a.y, b.y), m2(a.z, b.z), m2(a.w, b.w)); }
};

// masks (optional): the layer's per-tile reuse bitmaps; a pixel whose bit is set was filled from the cache
template <typename T>
__global__ void k_maxpool_vec(const T* in, int Hi, int Wi, int C, int S, dc_layer_desc L, T* out, const uint32_t* masks,
                              int tiles_x, int tiles_y)
{
    constexpr int N = Vec16<T>::N;
    const int cv = C / N;
    const size_t total = (size_t)S * L.out_h * L.out_w * cv;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        int c = (int)(i % cv); size_t t = i / cv;
        int ox = (int)(t % L.out_w); t /= L.out_w;
        int oy = (int)(t % L.out_h); int s = (int)(t / L.out_h);
        if (masks) {
            const size_t tile = ((size_t)s * tiles_y + oy / DC_TILE_H) * tiles_x + ox / DC_TILE_W;
            const int bit = DC_TILE_BIT(oy % DC_TILE_H, ox % DC_TILE_W);
            if ((masks[tile * 4 + (bit >> 5)] >> (bit & 31)) & 1u) continue;
        }
        uint4 m = make_uint4(0, 0, 0, 0);
        bool first = true;
        for (int ky = 0; ky < L.kh; ++ky) {
            int iy = oy * L.sh - L.ph + ky;
            if (iy < 0 || iy >= Hi) continue;
            for (int kx = 0; kx < L.kw; ++kx) {
                int ix = ox * L.sw - L.pw + kx;
                if (ix < 0 || ix >= Wi) continue;
                uint4 v = __ldg((const uint4*)(in + (((size_t)s * Hi + iy) * Wi + ix) * C) + c);
                m = first ? v : Vec16<T>::vmax(m, v);
                first = false;
            }
        }
        *((uint4*)(out + i / cv * C) + c) = m;
    }
}

// 2 x 2 windows at stride 2 without padding (every window inside the map), no reuse bitmap: the four 16-byte
// loads of an output vector are independent and issued together; 32-bit index arithmetic.
template <typename T>
__global__ void k_maxpool2x2_vec(const uint4* in, int Hi, int Wi, int cv, int out_h, int out_w, unsigned total, uint4* out)
{
    for (unsigned i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
        const unsigned c = i % cv, t = i / cv, ox = t % out_w, u = t / out_w, oy = u % out_h, s = u / out_h;
        const uint4* p = in + (((size_t)s * Hi + 2 * oy) * Wi + 2 * ox) * cv + c;
        const size_t row = (size_t)Wi * cv;
        const uint4 v00 = __ldg(p), v01 = __ldg(p + cv), v10 = __ldg(p + row), v11 = __ldg(p + row + cv);
        out[i] = Vec16<T>::vmax(Vec16<T>::vmax(v00, v01), Vec16<T>::vmax(v10, v11));
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

// 16-byte vectors: element-wise add (+ ReLU) and ReLU are pure HBM traffic, one vector per thread and pass
template <typename T> struct VecOps;
template <> struct VecOps<float> {
    static __device__ __forceinline__ uint4 add(uint4 a, uint4 b, int relu)
    {
        float r[4] = {__uint_as_float(a.x) + __uint_as_float(b.x), __uint_as_float(a.y) + __uint_as_float(b.y),
                      __uint_as_float(a.z) + __uint_as_float(b.z), __uint_as_float(a.w) + __uint_as_float(b.w)};
        if (relu) { for (int i = 0; i < 4; ++i) r[i] = fmaxf(r[i], 0.f); }
        return make_uint4(__float_as_uint(r[0]), __float_as_uint(r[1]), __float_as_uint(r[2]), __float_as_uint(r[3]));
    }
};
template <> struct VecOps<__nv_bfloat16> {
    static __device__ __forceinline__ uint32_t add2(uint32_t a, uint32_t b, int relu)
    {
        const float2 fa = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&a));
        const float2 fb = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&b));
        float x = fa.x + fb.x, y = fa.y + fb.y;                   // fp32 sum, one rounding to bf16 (as the scalar kernel)
        if (relu) { x = fmaxf(x, 0.f); y = fmaxf(y, 0.f); }
        __nv_bfloat162 r = __floats2bfloat162_rn(x, y);
        return *reinterpret_cast<uint32_t*>(&r);
    }
    static __device__ __forceinline__ uint4 add(uint4 a, uint4 b, int relu)
    {
        return make_uint4(add2(a.x, b.x, relu), add2(a.y, b.y, relu), add2(a.z, b.z, relu), add2(a.w, b.w, relu));
    }
};

// out = a + b (+ ReLU); with b == nullptr: out = ReLU(a) (a + 0 is exact)
template <typename T>
__global__ void k_add_vec(const uint4* a, const uint4* b, size_t nvec, int relu, uint4* out)
{
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += (size_t)gridDim.x * blockDim.x) {
        const uint4 va = __ldg(a + i), vb = b ? __ldg(b + i) : make_uint4(0, 0, 0, 0);
        out[i] = VecOps<T>::add(va, vb, relu);
    }
}

// Local response normalisation inside each channel over a (2 r + 1)^2 window; pixels outside the map count as zero
// and the divisor stays n^2 at the borders.  One thread per output element; sums in float.
template <typename T>
__global__ void k_lrn(const T* in, int H, int W, int C, int S, int r, float alpha_n2, float beta, float kappa, T* out,
                      const uint32_t* masks, int tiles_x, int tiles_y)
{
    const size_t total = (size_t)S * H * W * C;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int c = (int)(i % C); size_t t = i / C;
        const int x = (int)(t % W); t /= W;
        const int y = (int)(t % H); const int s = (int)(t / H);
        if (masks) {                                             // pixel filled from the cache
            const size_t tile = ((size_t)s * tiles_y + y / DC_TILE_H) * tiles_x + x / DC_TILE_W;
            const int bit = DC_TILE_BIT(y % DC_TILE_H, x % DC_TILE_W);
            if ((masks[tile * 4 + (bit >> 5)] >> (bit & 31)) & 1u) continue;
        }
        float sum = 0.f;
        for (int dy = -r; dy <= r; ++dy) {
            const int yy = y + dy;
            if (yy < 0 || yy >= H) continue;
            for (int dx = -r; dx <= r; ++dx) {
                const int xx = x + dx;
                if (xx < 0 || xx >= W) continue;
                const float v = to_f(in[(((size_t)s * H + yy) * W + xx) * C + c]);
                sum += v * v;
            }
        }
        out[i] = from_f<T>(to_f(in[i]) * powf(kappa + alpha_n2 * sum, -beta));
    }
}

// Channel concatenation of two NHWC maps
template <typename T>
__global__ void k_concat(const T* a, int Ca, const T* b, int Cb, size_t pixels, T* out)
{
    const int C = Ca + Cb;
    const size_t total = pixels * C;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int c = (int)(i % C); const size_t px = i / C;
        out[i] = c < Ca ? a[px * Ca + c] : b[px * Cb + (c - Ca)];
    }
}

inline int grid_for(const dc_cache* c, size_t n, int block)
{
    const size_t g = (n + block - 1) / block, cap = (size_t)c->num_sms * 16;
    return (int)(g > cap ? cap : (g ? g : 1));
}

}  // namespace

#define DISPATCH(c, expr_f32, expr_bf16) do { if ((c)->cfg.dtype == DC_BF16) { expr_bf16; } else { expr_f32; } } while (0)

int dc_launch_input_map(dc_cache* c, const uint8_t* frame, size_t pitch)
{
    size_t n = (size_t)c->S * c->cfg.height * c->cfg.width * 3;
    int W = c->cfg.width, H = c->cfg.height;
    dc_prof_scope ps(c, DC_ST_INPUT);
    DISPATCH(c,
        (k_input_map<float><<<grid_for(c, n, 256), 256, 0, c->stream>>>(frame, pitch, W, H, c->S, (const float*)c->pix_lut, (float*)c->input_map)),
        (k_input_map<__nv_bfloat16><<<grid_for(c, n, 256), 256, 0, c->stream>>>(frame, pitch, W, H, c->S, (const __nv_bfloat16*)c->pix_lut, (__nv_bfloat16*)c->input_map)));
    c->launches += 1;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}

int dc_launch_resize(dc_cache* c, int layer, const uint8_t* frame, size_t pitch)
{
    dc_layer_rt& L = c->L[layer];
    int grid = c->S * L.d.out_h;
    size_t smem = (size_t)((c->cfg.width * 3 + 15) / 16) * 16 * sizeof(uint16_t);
    if (smem > 48 * 1024 || (size_t)c->cfg.height > 255u * (size_t)L.d.out_h) return DC_ERR_CONFIG;   // 16-bit column sums
    dc_prof_scope ps(c, DC_ST_INPUT);
    DISPATCH(c,
        (k_resize_area<float><<<grid, 256, smem, c->stream>>>(frame, pitch, c->cfg.width, c->cfg.height, c->S, L.d.out_w, L.d.out_h, (float*)L.map[0])),
        (k_resize_area<__nv_bfloat16><<<grid, 256, smem, c->stream>>>(frame, pitch, c->cfg.width, c->cfg.height, c->S, L.d.out_w, L.d.out_h, (__nv_bfloat16*)L.map[0])));
    c->launches += 1;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}

int dc_launch_maxpool(dc_cache* c, int layer, const void* in, void* out, const uint32_t* masks)
{
    dc_layer_rt& L = c->L[layer];
    size_t n = (size_t)c->S * L.d.out_h * L.d.out_w * L.d.cout;
    dc_prof_scope ps(c, DC_ST_POINTWISE);
    if ((L.d.cout * c->elt) % 16 == 0 && !masks && L.d.kh == 2 && L.d.kw == 2 && L.d.sh == 2 && L.d.sw == 2 && L.d.ph == 0 &&
        L.d.pw == 0 && 2 * L.d.out_h <= L.in_h && 2 * L.d.out_w <= L.in_w && n * c->elt / 16 < 0x7fffffffull) {
        const unsigned nv = (unsigned)(n * c->elt / 16);
        const int cv = L.d.cout * c->elt / 16;
        DISPATCH(c,
            (k_maxpool2x2_vec<float><<<grid_for(c, nv, 256), 256, 0, c->stream>>>((const uint4*)in, L.in_h, L.in_w, cv, L.d.out_h, L.d.out_w, nv, (uint4*)out)),
            (k_maxpool2x2_vec<__nv_bfloat16><<<grid_for(c, nv, 256), 256, 0, c->stream>>>((const uint4*)in, L.in_h, L.in_w, cv, L.d.out_h, L.d.out_w, nv, (uint4*)out)));
        c->launches += 1;
        DC_CUDA(cudaGetLastError());
        return DC_OK;
    }
    if ((L.d.cout * c->elt) % 16 == 0) {
        size_t nv = n * c->elt / 16;
        DISPATCH(c,
            (k_maxpool_vec<float><<<grid_for(c, nv, 256), 256, 0, c->stream>>>((const float*)in, L.in_h, L.in_w, L.d.cout, c->S, L.d, (float*)out, masks, L.tiles_x, L.tiles_y)),
            (k_maxpool_vec<__nv_bfloat16><<<grid_for(c, nv, 256), 256, 0, c->stream>>>((const __nv_bfloat16*)in, L.in_h, L.in_w, L.d.cout, c->S, L.d, (__nv_bfloat16*)out, masks, L.tiles_x, L.tiles_y)));
        c->launches += 1;
        DC_CUDA(cudaGetLastError());
        return DC_OK;
    }
    if (masks) return DC_ERR_STATE;                             // cached pooling needs 16-byte pixels (checked at creation)
    DISPATCH(c,
        (k_maxpool<float><<<grid_for(c, n, 256), 256, 0, c->stream>>>((const float*)in, L.in_h, L.in_w, L.d.cout, c->S, L.d, (float*)out)),
        (k_maxpool<__nv_bfloat16><<<grid_for(c, n, 256), 256, 0, c->stream>>>((const __nv_bfloat16*)in, L.in_h, L.in_w, L.d.cout, c->S, L.d, (__nv_bfloat16*)out)));
    c->launches += 1;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}

int dc_launch_add(dc_cache* c, int layer, const void* a, const void* b)
{
    dc_layer_rt& L = c->L[layer];
    size_t n = (size_t)c->S * L.d.out_h * L.d.out_w * L.d.cout;
    dc_prof_scope ps(c, DC_ST_POINTWISE);
    if ((n * c->elt) % 16 == 0) {                                 // maps come from cudaMalloc: 256-byte aligned
        const size_t nv = n * c->elt / 16;
        DISPATCH(c,
            (k_add_vec<float><<<grid_for(c, nv, 256), 256, 0, c->stream>>>((const uint4*)a, (const uint4*)b, nv, L.d.relu, (uint4*)L.map[0])),
            (k_add_vec<__nv_bfloat16><<<grid_for(c, nv, 256), 256, 0, c->stream>>>((const uint4*)a, (const uint4*)b, nv, L.d.relu, (uint4*)L.map[0])));
    } else {
        DISPATCH(c,
            (k_add<float><<<grid_for(c, n, 256), 256, 0, c->stream>>>((const float*)a, (const float*)b, n, L.d.relu, (float*)L.map[0])),
            (k_add<__nv_bfloat16><<<grid_for(c, n, 256), 256, 0, c->stream>>>((const __nv_bfloat16*)a, (const __nv_bfloat16*)b, n, L.d.relu, (__nv_bfloat16*)L.map[0])));
    }
    c->launches += 1;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}

int dc_launch_relu(dc_cache* c, int layer, const void* a)
{
    dc_layer_rt& L = c->L[layer];
    size_t n = (size_t)c->S * L.d.out_h * L.d.out_w * L.d.cout;
    dc_prof_scope ps(c, DC_ST_POINTWISE);
    if ((n * c->elt) % 16 == 0) {
        const size_t nv = n * c->elt / 16;
        DISPATCH(c,
            (k_add_vec<float><<<grid_for(c, nv, 256), 256, 0, c->stream>>>((const uint4*)a, nullptr, nv, 1, (uint4*)L.map[0])),
            (k_add_vec<__nv_bfloat16><<<grid_for(c, nv, 256), 256, 0, c->stream>>>((const uint4*)a, nullptr, nv, 1, (uint4*)L.map[0])));
    } else {
        DISPATCH(c,
            (k_relu<float><<<grid_for(c, n, 256), 256, 0, c->stream>>>((const float*)a, n, (float*)L.map[0])),
            (k_relu<__nv_bfloat16><<<grid_for(c, n, 256), 256, 0, c->stream>>>((const __nv_bfloat16*)a, n, (__nv_bfloat16*)L.map[0])));
    }
    c->launches += 1;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}

int dc_launch_lrn(dc_cache* c, int layer, const void* in, void* out, const uint32_t* masks)
{
    dc_layer_rt& L = c->L[layer];
    const size_t n = (size_t)c->S * L.d.out_h * L.d.out_w * L.d.cout;
    const int r = L.d.ph, win = 2 * r + 1;
    const bool defaults = c->cfg.lrn_alpha == 0.0 && c->cfg.lrn_beta == 0.0 && c->cfg.lrn_k == 0.0;
    const float alpha = (float)(defaults ? 1e-4 : c->cfg.lrn_alpha), beta = (float)(defaults ? 0.75 : c->cfg.lrn_beta);
    const float kappa = (float)(defaults ? 1.0 : c->cfg.lrn_k);
    dc_prof_scope ps(c, DC_ST_POINTWISE);
    DISPATCH(c,
        (k_lrn<float><<<grid_for(c, n, 256), 256, 0, c->stream>>>((const float*)in, L.d.out_h, L.d.out_w, L.d.cout, c->S, r, alpha / (win * win), beta, kappa, (float*)out, masks, L.tiles_x, L.tiles_y)),
        (k_lrn<__nv_bfloat16><<<grid_for(c, n, 256), 256, 0, c->stream>>>((const __nv_bfloat16*)in, L.d.out_h, L.d.out_w, L.d.cout, c->S, r, alpha / (win * win), beta, kappa, (__nv_bfloat16*)out, masks, L.tiles_x, L.tiles_y)));
    c->launches += 1;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}

int dc_launch_concat(dc_cache* c, int layer, const void* a, int ca, const void* b, int cb)
{
    dc_layer_rt& L = c->L[layer];
    const size_t pixels = (size_t)c->S * L.d.out_h * L.d.out_w;
    dc_prof_scope ps(c, DC_ST_POINTWISE);
    DISPATCH(c,
        (k_concat<float><<<grid_for(c, pixels * L.d.cout, 256), 256, 0, c->stream>>>((const float*)a, ca, (const float*)b, cb, pixels, (float*)L.map[0])),
        (k_concat<__nv_bfloat16><<<grid_for(c, pixels * L.d.cout, 256), 256, 0, c->stream>>>((const __nv_bfloat16*)a, ca, (const __nv_bfloat16*)b, cb, pixels, (__nv_bfloat16*)L.map[0])));
    c->launches += 1;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}
