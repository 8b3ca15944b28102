// Strided convolutions over few input channels (a network's first layer: 11 x 11 stride 4 or 7 x 7 stride 2 on RGB)
// as stride-1 convolutions over a space-to-depth copy of the input.
//
// A convolution with stride s reads, for neighbouring output pixels, input pixels s apart: no operand scheme of the
// tensor-core kernels can reuse a fetched window across taps, and with three channels a tap is a sliver of K.  Cut the
// (padded) input into s x s blocks and make every block one pixel of s * s * cin channels: output pixel (oy, ox) then
// needs the blocks (oy + ty, ox + tx), ty < Ty, tx < Tx - a stride-1 convolution without padding whose kernel has
// Ty x Tx taps of s * s * cin channels each (weights that fall outside the original kernel are zero).  With
//     Py = ceil(ph / s) * s   rows of zeros in front of the input (so that blocks start on multiples of s),
//     offy = Py - ph,   Ty = ceil((kh + offy) / s),   block map height Ho + Ty - 1        (columns alike)
// the original tap ky of output row oy reads input row oy * s - ph + ky = (oy + ty) * s + dy - Py with
// ky + offy = ty * s + dy.  The sums are the same products in another order plus zeros; the layer's output, its
// rectangles (Table 2 works on the layer as declared) and its tiles do not change.
//
// The rewritten layer (channels padded to 16, 32 or 64) runs on the ordinary kernels: AlexNet's first layer becomes a
// 3 x 3 convolution over 64 channels (column slabs), ResNet's stem a 4 x 4 convolution over 16.  (The same rewrite with
// 1 x 1 blocks, padding a stride-1 layer's 96 channels to 128 so that it leaves the tap-by-tap kernel, was measured on
// AlexNet's second layer: faster alone, slower in the trunk with the copy it needs: not kept.)
#include "dc_common.cuh"

#include <cuda_bf16.h>
#include <cstdlib>

namespace {

struct S2dArgs {
    const __nv_bfloat16* in; __nv_bfloat16* out;
    int S, Hi, Wi, cin, s, Py, Px, Hs, Ws, cs;      // cs: channels of a block pixel (padded)
};

// One thread per 8 channels (16 bytes) of a block pixel.
__global__ void k_space_to_depth(const S2dArgs a)
{
    const int chunks = a.cs / 8;
    const size_t total = (size_t)a.S * a.Hs * a.Ws * chunks;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        size_t r = i;
        const int ch = (int)(r % chunks); r /= chunks;
        const int bx = (int)(r % a.Ws); r /= a.Ws;
        const int by = (int)(r % a.Hs);
        const int st = (int)(r / a.Hs);
        const __nv_bfloat16* src = a.in + (size_t)st * a.Hi * a.Wi * a.cin;
        __align__(16) __nv_bfloat16 v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int e = ch * 8 + j, q = e / a.cin, cc = e - q * a.cin;      // q: which pixel of the s x s block
            const int dy = q / a.s, dx = q - dy * a.s;
            const int iy = by * a.s + dy - a.Py, ix = bx * a.s + dx - a.Px;
            const bool on = q < a.s * a.s && iy >= 0 && iy < a.Hi && ix >= 0 && ix < a.Wi;
            v[j] = on ? src[((size_t)iy * a.Wi + ix) * a.cin + cc] : __float2bfloat16(0.f);
        }
        *(uint4*)(a.out + i * 8) = *(const uint4*)v;
    }
}

// w [cout][kh][kw][cin] -> w' [cout][Ty][Tx][cs]
__global__ void k_s2d_weights(const __nv_bfloat16* w, int cout, int kh, int kw, int cin, int s, int offy, int offx, int Ty, int Tx, int cs,
                              __nv_bfloat16* out)
{
    const size_t total = (size_t)cout * Ty * Tx * cs;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        size_t r = i;
        const int e = (int)(r % cs); r /= cs;
        const int tx = (int)(r % Tx); r /= Tx;
        const int ty = (int)(r % Ty);
        const int co = (int)(r / Ty);
        const int q = e / cin, cc = e - q * cin, dy = q / s, dx = q - dy * s;
        const int ky = ty * s + dy - offy, kx = tx * s + dx - offx;
        const bool on = q < s * s && ky >= 0 && ky < kh && kx >= 0 && kx < kw;
        out[i] = on ? w[(((size_t)co * kh + ky) * kw + kx) * cin + cc] : __float2bfloat16(0.f);
    }
}

}  // namespace

// Whether `d` (a layer as declared) is rewritten: a strided convolution whose s x s blocks fit 64 channels.
// DC_NO_S2D=1 (diagnostics) keeps every layer as declared.
bool dc_s2d_eligible(const dc_cache* c, const dc_layer_desc& d)
{
    if (c->cfg.dtype != DC_BF16 || !c->executable || getenv("DC_NO_S2D") || getenv("DC_NO_TENSOR_CORES")) return false;
    if (d.kind != DC_CONV || d.groups > 1 || d.sh != d.sw || d.sh < 2 || d.sh > 8 || d.cout % 32 != 0) return false;
    if (d.cin * d.sh * d.sw > 64) return false;
    const int s = d.sh;
    const int offy = (d.ph + s - 1) / s * s - d.ph, offx = (d.pw + s - 1) / s * s - d.pw;
    return (d.kh + offy + s - 1) / s <= 5 && (d.kw + offx + s - 1) / s <= 5;      // what every operand scheme takes
}

// Called once per eligible layer, after its weights exist in [cout][kh][kw][cin] bf16: replaces them by the
// rewritten layer's, allocates the block map and rewrites the layer as the kernels see it.
int dc_s2d_rewrite(dc_cache* c, int layer)
{
    dc_layer_rt& L = c->L[layer];
    const dc_layer_desc d = L.d;
    const int s = d.sh;
    const int Py = (d.ph + s - 1) / s * s, Px = (d.pw + s - 1) / s * s;
    const int offy = Py - d.ph, offx = Px - d.pw;
    const int Ty = (d.kh + offy + s - 1) / s, Tx = (d.kw + offx + s - 1) / s;
    // block pixels padded to 16, 32 or 64 channels, whichever holds them (always 64, so that the stem of ResNet could run
    // on column slabs, was measured: the same 0.21 ms for the layer, and a block map four times the size)
    const int cb = d.cin * s * s, cs = cb <= 16 ? 16 : cb <= 32 ? 32 : 64;
    const int Hs = d.out_h + Ty - 1, Ws = d.out_w + Tx - 1;
    const size_t wn = (size_t)d.cout * Ty * Tx * cs, mn = (size_t)c->S * Hs * Ws * cs;
    void* w2 = nullptr;
    DC_CUDA(cudaMalloc(&w2, wn * 2));
    DC_CUDA(cudaMalloc(&L.in_s2d, mn * 2));
    c->bytes += wn * 2 + mn * 2;
    int grid = (int)((wn + 255) / 256); if (grid > c->num_sms * 8) grid = c->num_sms * 8;
    k_s2d_weights<<<grid, 256, 0, c->stream>>>((const __nv_bfloat16*)L.weight, d.cout, d.kh, d.kw, d.cin, s, offy, offx, Ty, Tx, cs,
                                               (__nv_bfloat16*)w2);
    DC_CUDA(cudaGetLastError());
    DC_CUDA(cudaMemsetAsync(L.in_s2d, 0, mn * 2, c->stream));
    DC_CUDA(cudaStreamSynchronize(c->stream));                   // the old weights are read by the kernel above
    const size_t old_bytes = (size_t)d.cout * d.kh * d.kw * d.cin * 2;
    cudaFree(L.weight);
    c->bytes -= old_bytes;
    L.weight = w2;
    L.s2d_s = s; L.s2d_py = Py; L.s2d_px = Px; L.s2d_cin = d.cin; L.s2d_hi = L.in_h; L.s2d_wi = L.in_w;
    L.d.kh = Ty; L.d.kw = Tx; L.d.sh = L.d.sw = 1; L.d.ph = L.d.pw = 0; L.d.cin = cs;
    L.in_h = Hs; L.in_w = Ws;
    return DC_OK;
}

// Fills the layer's block map from its input as declared ([S][Hi][Wi][cin] bf16).
int dc_launch_s2d(dc_cache* c, int layer, const void* in)
{
    dc_layer_rt& L = c->L[layer];
    S2dArgs a;
    a.in = (const __nv_bfloat16*)in; a.out = (__nv_bfloat16*)L.in_s2d;
    a.S = c->S; a.Hi = L.s2d_hi; a.Wi = L.s2d_wi; a.cin = L.s2d_cin; a.s = L.s2d_s; a.Py = L.s2d_py; a.Px = L.s2d_px;
    a.Hs = L.in_h; a.Ws = L.in_w; a.cs = L.d.cin;
    const size_t total = (size_t)a.S * a.Hs * a.Ws * (a.cs / 8);
    int grid = (int)((total + 255) / 256); if (grid > c->num_sms * 16) grid = c->num_sms * 16;
    k_space_to_depth<<<grid, 256, 0, c->stream>>>(a);
    c->launches += 1;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}
