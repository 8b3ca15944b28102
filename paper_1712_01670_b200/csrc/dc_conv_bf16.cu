// Partial convolution on the 5th-generation tensor cores (bf16 in, fp32 accumulate in TMEM).
//
// Section 5, "Reuse", third step: convolve only what the cache did not supply.  The unit of
// work is one dirty 16x8 output tile (128 pixels = the M of one tcgen05.mma) times one block of
// BN output channels.  It is an implicit GEMM: for every kernel tap (ky, kx) and every chunk of
// BK input channels, TMA fetches
//     A: the 16x8 window of the NHWC input map displaced by the tap (a 4-D box; coordinates
//        outside the map are zero-filled, which is the convolution's padding), 128 rows x BK
//     B: BN rows x BK of the weights, which are already K-major as [cout][kh][kw][cin]
// into 128-byte-swizzled shared memory, and one elected thread issues BK/16 tcgen05.mma
// (M = 128, N = BN, K = 16) accumulating into tensor memory.
//
// Warp roles in a CTA of 192 threads (persistent, one CTA per SM):
//     warp 0      TMA producer             (full/empty mbarrier ring of `stages` slots)
//     warp 1      TMEM allocation, MMA issue, tcgen05.commit
//     warps 2-5   epilogue: tcgen05.ld of their 32-lane quadrant, + bias, ReLU, bf16, and a
//                 store predicated on the tile's reuse bitmap (only non-reused pixels are written)
// Two accumulators (2 x BN TMEM columns) let the epilogue of one work item overlap the MMAs of
// the next.  Every mbarrier wait is bounded: on expiry the kernel records DC_ERR_TIMEOUT in the
// status word, all roles leave their loops, tensor memory is freed and the kernel returns.
#include <cuda.h>
#include <stdio.h>
#include <stdlib.h>

#include "dc_common.cuh"

namespace {

constexpr int kThreads = 192;          // producer warp, MMA warp, four epilogue warps
constexpr int kThreadsWide = 320;      // ... or eight epilogue warps
static inline int threads_for(int epi_warps) { return 64 + 32 * epi_warps; }
constexpr int kMaxStages = 8;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // 2 s

struct TcArgs {
    const float* bias; __nv_bfloat16* out;
    const int32_t* tile_list; const int32_t* tile_count; const uint32_t* masks;
    int Ho, Wo, Co, Ci, kh, kw, sh, sw, ph, pw, relu, tiles_x, tiles_y;
    int BN, NB, BK, kchunks, stages, a_bytes, b_bytes;
    int nb_off;                   // grouped convolution: first channel block of the group this launch computes
    int MT, nbuf;                 // tiles per work item (1 or 2, sharing one B tile); TMEM accumulator sets (2, or 1 when MT * BN = 512)
    uint32_t idesc, sbo, layout_type;
    uint32_t tmem_cols;           // TMEM columns this CTA allocates: a power of two >= nbuf * MT * BN (256 at most when two CTAs share an SM)
    int32_t* status;
    unsigned long long wait_ns;   // limit of every device-side wait
    int skip_loads;               // failure-detection tests: the producer issues no copy, so the other roles' waits run out
    // flat tiles (tap-by-tap kernel only): row i of tile t is group t * 16 + i, a group being 8 output pixels of one
    // image row, numbered (stream * Ho + y) * gpr + column group; n_groups_all = S * Ho * gpr.  0: 16 x 8 blocks.
    int flat = 0, gpr = 0, n_groups_all = 0;
    int epi_warps = 4;            // epilogue warps of the CTA: 4 (192 threads) or 8 (320 threads)
    int bias_smem = 0;            // > 0: that many bias values (the launch's NB * BN, from channel block nb_off on) are staged in shared memory behind the control block
};

struct SmemCtl {
    unsigned long long full[kMaxStages], empty[kMaxStages], tmem_full[2], tmem_empty[2];
    unsigned long long a_full[4], a_empty[4];     // halo kernel: ring of input patches
    uint32_t tmem_base;
    volatile int abort_flag;
    unsigned long long wait_ns;
    // epilogue staging: per warp 32 pixels x 64 bytes (32 bf16 channels), rows padded to 80 bytes so
    // 16-byte accesses of neighbouring lanes fall in different banks.  Last member: a launch with four epilogue
    // warps asks for (and touches) the first four only, see ctl_bytes().
    __align__(16) uint8_t stage[8][32 * 80];
};
constexpr int kStageBytes = 32 * 80;
// Shared memory the control block takes with `epi_warps` epilogue warps (4 or 8).
__host__ __device__ constexpr size_t ctl_bytes(int epi_warps) { return sizeof(SmemCtl) - (size_t)(8 - epi_warps) * kStageBytes; }

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Programmatic dependent launch: a convolution kernel is launched so that its CTAs may become resident while the
// previous kernel of the stream is still running (on SMs that kernel has left).  Barrier set-up, tensor-memory
// allocation and descriptor prefetch run there; pdl_wait() returns once the previous kernel has completed and its
// writes are visible, and nothing that another kernel produces is read (or overwritten) before it.
// pdl_release() lets the kernel after this one do the same.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void mbar_init(void* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(void* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(void* bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Arrival that orders nothing but the barrier itself: used to hand a TMEM accumulator back (its reads are
// ordered by tcgen05.wait::ld + tcgen05.fence), so the arrival need not wait for the epilogue's global stores.
__device__ __forceinline__ void mbar_arrive_relaxed(void* bar)
{
    asm volatile("mbarrier.arrive.relaxed.cta.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Arrival on a barrier in the other CTA of a pair (addr: shared::cluster address from mapa).
__device__ __forceinline__ void mbar_arrive_remote(uint32_t addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(addr) : "memory");
}
__device__ __forceinline__ bool mbar_try(void* bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long now_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait.  Returns false (and raises the abort flag + status word) when the limit passes
// or another role has already given up.
__device__ __forceinline__ bool mbar_wait(void* bar, uint32_t parity, SmemCtl* ctl, int32_t* status)
{
    if (mbar_try(bar, parity)) return true;
    const unsigned long long t0 = now_ns();
    for (uint32_t spin = 1;; ++spin) {
        if (mbar_try(bar, parity)) return true;
        if ((spin & 255u) == 0) {
            if (ctl->abort_flag) return false;
            if (now_ns() - t0 > ctl->wait_ns) {
                ctl->abort_flag = 1;
                atomicExch(status, (int)DC_ERR_TIMEOUT);
                return false;
            }
        }
    }
}

__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* tm, int c0, int c1, int c2, int c3, void* bar)
{
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
                 ::"r"(smem_u32(dst)), "l"(tm), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* tm, int c0, int c1, void* bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(smem_u32(dst)), "l"(tm), "r"(smem_u32(bar)), "r"(c0), "r"(c1) : "memory");
}

// K-major operand tile in shared memory.  Swizzled layouts: rows of BK bf16, 8-row groups `sbo`
// bytes apart (lbo unused, 16).  Unswizzled layout (layout_type 0): 8-row x 16-byte core matrices,
// `sbo` bytes apart along M/N and `lbo` bytes apart along K.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t sbo, uint32_t layout_type, uint32_t lbo = 16)
{
    uint32_t lo = ((saddr >> 4) & 0x3FFFu) | (((lbo >> 4) & 0x3FFFu) << 16);   // start address, LBO
    uint32_t hi = ((sbo >> 4) & 0x3FFFu) | (1u << 14) | (layout_type << 29);   // SBO, descriptor version 1, swizzle
    return ((uint64_t)hi << 32) | lo;
}
__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(void* bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r)
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ uint32_t pack_bf16(float a, float b)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&v);
}
// 16-byte accesses to the epilogue's staging by shared-space address: through a generic pointer they would be
// generic loads and stores, which resolve the address space first and wait on the long-latency scoreboard.
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t x, uint32_t y, uint32_t z, uint32_t w)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
// (acc0 + b0, acc1 + b1) in fp32 (one packed add), then round to nearest even into two bf16; RELU clamps negative
// results to zero in the same conversion (rounding is monotonic, so clamping before or after it gives the same value).
template <bool RELU>
__device__ __forceinline__ uint32_t bias_pack_bf16(uint32_t acc0, uint32_t acc1, float b0, float b1)
{
    uint32_t out;
    if (RELU)
        asm("{\n\t.reg .b64 a, b, d;\n\t.reg .f32 x, y;\n\tmov.b64 a, {%1, %2};\n\tmov.b64 b, {%3, %4};\n\t"
            "add.rn.f32x2 d, a, b;\n\tmov.b64 {x, y}, d;\n\tcvt.rn.relu.bf16x2.f32 %0, y, x;\n\t}"
            : "=r"(out) : "r"(acc0), "r"(acc1), "f"(b0), "f"(b1));
    else
        asm("{\n\t.reg .b64 a, b, d;\n\t.reg .f32 x, y;\n\tmov.b64 a, {%1, %2};\n\tmov.b64 b, {%3, %4};\n\t"
            "add.rn.f32x2 d, a, b;\n\tmov.b64 {x, y}, d;\n\tcvt.rn.bf16x2.f32 %0, y, x;\n\t}"
            : "=r"(out) : "r"(acc0), "r"(acc1), "f"(b0), "f"(b1));
    return out;
}

// Copies the launch's bias values behind the control block (all threads; before the set-up's __syncthreads).  The
// epilogue reads 32 of them per step and lane: from shared memory that is eight short broadcast loads, through the
// read-only cache it was a fifth of the time of the layers that the epilogue bounds.
__device__ __forceinline__ void stage_bias(const TcArgs& a, SmemCtl* ctl, int epi_warps)
{
    float* dst = (float*)((uint8_t*)ctl + ctl_bytes(epi_warps));
    const float* src = a.bias + (size_t)a.nb_off * a.BN;
    for (int i = threadIdx.x; i < a.bias_smem; i += blockDim.x) dst[i] = __ldg(src + i);
}

// Epilogue warps (4 warps = 128 TMEM lanes = the 128 pixels of a tile): for every work item wait
// for its accumulator, read it 32 columns at a time, add the bias, apply ReLU, round to bf16 and
// store the pixel's channels unless the reuse bitmap says the pixel was filled from the cache.
// epi_warps = 8: two warps per TMEM lane quadrant (warps 2-5 and 6-9), each taking half of the item's channels:
// layers with little accumulation per output (1x1, few input channels) are bound by this read-out.
// first_item / item_stride: the items this CTA (or CTA pair) takes.  tiles_per_group / tile_sub: a group of the tile list
// holds tiles_per_group tiles and this CTA's first one is number tile_sub in it (a pair: 2 and its rank, with a.MT = 1).
// remote_empty: 0, or the shared::cluster address of the pair leader's tmem_empty[0], on which this CTA's epilogue
// threads arrive instead of on their own.
__device__ __forceinline__ void epilogue_loop(const TcArgs& a, SmemCtl* ctl, uint32_t tmem_base, int n_items, int n_tiles, int warp, int lane,
                                              int first_item, int item_stride, int tiles_per_group, int tile_sub, uint32_t remote_empty,
                                              int epi_warps = 4)
{
    // the launch's bias values in shared memory (stage_bias), or 0: read through the read-only cache
    const uint32_t bias_s = a.bias_smem > 0 ? smem_u32((const uint8_t*)ctl + ctl_bytes(epi_warps)) : 0u;
    const int per_stream = a.tiles_x * a.tiles_y;
    const int q = warp & 3;                                     // TMEM lane quadrant this warp may read
    // this warp's 32-column steps of an item: all of them, or the lower / upper half
    const int n_steps = a.BN / 32, mid = epi_warps == 8 ? (n_steps + 1) / 2 : n_steps;
    const int c_begin = warp >= 6 ? mid : 0, c_end = warp >= 6 ? n_steps : mid;
    const int m = q * 32 + lane, prow = m / DC_TILE_W, pcol = m % DC_TILE_W;
    const int mword_i = DC_TILE_BIT(prow, pcol) >> 5, mbit = DC_TILE_BIT(prow, pcol) & 31;
    uint32_t acc = 0, acc_ph = 0;
    bool ok = true;
    // the tile index and this pixel's bitmap word of the NEXT item are fetched while the current one is
    // processed: two dependent global loads would otherwise sit on every item's critical path
    int tile_n0 = -1, tile_n1 = -1; uint32_t mask_n0 = 0, mask_n1 = 0;       // scalars: indexed arrays would live in local memory
    auto fetch = [&](int item) {
        if (item >= n_items) return;
        const int idx = (item / a.NB) * tiles_per_group + tile_sub;
        tile_n0 = idx < n_tiles ? a.tile_list[idx] : -1;                           // a pair's second CTA may have no tile in the last group
        mask_n0 = tile_n0 >= 0 ? a.masks[(size_t)tile_n0 * 4 + mword_i] : 0u;
        tile_n1 = (a.MT > 1 && idx + 1 < n_tiles) ? a.tile_list[idx + 1] : -1;     // odd tile count: the last item has one tile
        mask_n1 = tile_n1 >= 0 ? a.masks[(size_t)tile_n1 * 4 + mword_i] : 0u;
    };
    fetch(first_item);
    for (int item = first_item; item < n_items && ok; item += item_stride) {
        const int nb = item % a.NB;
        const int tile_c0 = tile_n0, tile_c1 = tile_n1;
        const uint32_t mask_c0 = mask_n0, mask_c1 = mask_n1;
        fetch(item + item_stride);
        ok = mbar_wait(&ctl->tmem_full[acc], acc_ph, ctl, a.status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        const float* bias = a.bias + (nb + a.nb_off) * a.BN;
        for (int j = 0; j < a.MT; ++j) {
            const int tile = j == 0 ? tile_c0 : tile_c1;
            if (tile < 0) break;
            const bool reused = ((j == 0 ? mask_c0 : mask_c1) >> mbit) & 1u;
            bool active;
            // write-back addressing, once per tile: piece k of this lane is the 16-byte part (lane & 3) of the pixel in
            // tile row q * 4 + k, column lane >> 2 (the warp's 32 pixels are 4 tile rows of 8)
            const size_t row_stride = (size_t)a.Wo * a.Co;
            const size_t ch_off = (size_t)(nb + a.nb_off) * a.BN + (lane & 3) * 8;
            size_t wb_off[4];                                   // element offset of piece k's pixel
            if (a.flat) {
                const int gps = a.Ho * a.gpr;
                const int g = tile * DC_TILE_H + prow, s = g / gps, loc = g - s * gps, y = loc / a.gpr, gx = loc - y * a.gpr;
                active = g < a.n_groups_all && gx * DC_TILE_W + pcol < a.Wo && !reused;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int gk = tile * DC_TILE_H + q * 4 + k, sk = gk / gps, lk = gk - sk * gps, yk = lk / a.gpr, xk = lk - yk * a.gpr;
                    wb_off[k] = (((size_t)sk * a.Ho + yk) * a.Wo + xk * DC_TILE_W + (lane >> 2)) * a.Co + ch_off;
                }
            } else {
                const int s = tile / per_stream, t = tile - s * per_stream, ty = t / a.tiles_x, tx = t - ty * a.tiles_x;
                const int oy = ty * DC_TILE_H + prow, ox = tx * DC_TILE_W + pcol;
                active = oy < a.Ho && ox < a.Wo && !reused;
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    wb_off[k] = ((size_t)s * a.Ho + ty * DC_TILE_H + q * 4 + k) * row_stride + (size_t)(tx * DC_TILE_W + (lane >> 2)) * a.Co + ch_off;
            }
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (acc * (uint32_t)a.MT + (uint32_t)j) * (uint32_t)a.BN;
            // Each lane owns one pixel (TMEM lane) and gets 32 channels = 64 bytes per step.  Storing them
            // directly would make every warp store touch 32 different lines 16 bytes at a time (half-written
            // sectors); instead the warp stages its 32 x 64 bytes in shared memory and writes them back with
            // 4 lanes per pixel, so each pixel's 64 bytes leave as two whole sectors.
            const unsigned act_mask = __ballot_sync(0xffffffffu, active);
            const uint32_t stg = smem_u32(ctl->stage[warp - 2]);
            const uint32_t rd = stg + (lane >> 2) * 80 + (lane & 3) * 16, mine = stg + lane * 80;
            for (int c = c_begin; c < c_end; ++c) {
                uint32_t r[32];
                tmem_ld32(taddr + c * 32, r);
                // the step's 32 bias values travel while the accumulator read is in flight
                float4 bv[8];
                if (bias_s) {
                    const uint32_t b4 = bias_s + (uint32_t)(nb * a.BN + c * 32) * 4u;
#pragma unroll
                    for (int v = 0; v < 8; ++v) {
                        const uint4 t = lds128(b4 + v * 16);
                        bv[v] = make_float4(__uint_as_float(t.x), __uint_as_float(t.y), __uint_as_float(t.z), __uint_as_float(t.w));
                    }
                } else {
                    const float4* b4 = (const float4*)(bias + c * 32);
#pragma unroll
                    for (int v = 0; v < 8; ++v) bv[v] = __ldg(b4 + v);
                }
                tmem_ld_wait();
                if (a.relu) {
#pragma unroll
                    for (int v = 0; v < 4; ++v)
                        sts128(mine + v * 16, bias_pack_bf16<true>(r[v * 8 + 0], r[v * 8 + 1], bv[2 * v].x, bv[2 * v].y),
                               bias_pack_bf16<true>(r[v * 8 + 2], r[v * 8 + 3], bv[2 * v].z, bv[2 * v].w),
                               bias_pack_bf16<true>(r[v * 8 + 4], r[v * 8 + 5], bv[2 * v + 1].x, bv[2 * v + 1].y),
                               bias_pack_bf16<true>(r[v * 8 + 6], r[v * 8 + 7], bv[2 * v + 1].z, bv[2 * v + 1].w));
                } else {
#pragma unroll
                    for (int v = 0; v < 4; ++v)
                        sts128(mine + v * 16, bias_pack_bf16<false>(r[v * 8 + 0], r[v * 8 + 1], bv[2 * v].x, bv[2 * v].y),
                               bias_pack_bf16<false>(r[v * 8 + 2], r[v * 8 + 3], bv[2 * v].z, bv[2 * v].w),
                               bias_pack_bf16<false>(r[v * 8 + 4], r[v * 8 + 5], bv[2 * v + 1].x, bv[2 * v + 1].y),
                               bias_pack_bf16<false>(r[v * 8 + 6], r[v * 8 + 7], bv[2 * v + 1].z, bv[2 * v + 1].w));
                }
                __syncwarp();
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if ((act_mask >> ((lane >> 2) + 8 * k)) & 1u)
                        *(uint4*)(a.out + wb_off[k] + c * 32) = lds128(rd + k * (8 * 80));
                }
                __syncwarp();
            }
        }
        tc_fence_before();
        if (remote_empty) mbar_arrive_remote(remote_empty + acc * 8u);
        else mbar_arrive_relaxed(&ctl->tmem_empty[acc]);
        if (++acc == (uint32_t)a.nbuf) { acc = 0; acc_ph ^= 1u; }
    }
}

template <int MT>
__global__ void __launch_bounds__(kThreadsWide, 1)
k_conv_tc(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const TcArgs a)
{
    extern __shared__ uint8_t smem_raw[];

    // operand ring at a 1024-byte boundary (the swizzle pattern repeats every 1024 bytes), then control words
    uint8_t* ring = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int stage_bytes = MT * a.a_bytes + a.b_bytes;
    SmemCtl* ctl = (SmemCtl*)(ring + (size_t)a.stages * stage_bytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int per_stream = a.tiles_x * a.tiles_y;
    const int taps = a.kh * a.kw, kiters = taps * a.kchunks;

    if (threadIdx.x == 0) {
        for (int i = 0; i < a.stages; ++i) { mbar_init(&ctl->full[i], 1); mbar_init(&ctl->empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&ctl->tmem_full[i], 1); mbar_init(&ctl->tmem_empty[i], 32u * (uint32_t)a.epi_warps); }
        ctl->abort_flag = 0;
        ctl->wait_ns = a.wait_ns;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB) : "memory");
    }
    stage_bias(a, ctl, a.epi_warps);
    if (warp == 1) {       // up to 512 columns: two accumulators of up to 256 columns
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)), "r"(a.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    pdl_wait();                 // the previous kernel's output, the tile list and its count are read from here on
    pdl_release();
    const int n_tiles = *a.tile_count;
    const int n_items = (n_tiles + MT - 1) / MT * a.NB;     // an item: MT tiles x one block of BN channels; none for this CTA: it only frees its tensor memory

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        int st = 0; uint32_t ph = 0;                              // ring slot and its phase
        bool ok = true;
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
            const int group = item / a.NB, nb = item % a.NB;
            int sN[MT], xb[MT], yb[MT];
            // flat tiles: lane l fetches group (l & 15) of tile (l >> 4), one box of 8 pixels per tap and chunk
            int fs = 0, fx = 0, fy = 0; bool fon = false; uint32_t flat_tx = 0;
            if (a.flat) {
                const int j = lane >> 4, idx = group * MT + j;
                if (j < MT) {
                    const int tile = a.tile_list[idx < n_tiles ? idx : group * MT];
                    const int gps = a.Ho * a.gpr, g = tile * DC_TILE_H + (lane & 15);
                    fon = g < a.n_groups_all;                   // the last tile may have fewer groups: their rows stay as they are (never stored)
                    fs = g / gps;
                    const int loc = g - fs * gps, y = loc / a.gpr;
                    fx = (loc - y * a.gpr) * DC_TILE_W * a.sw - a.pw; fy = y * a.sh - a.ph;
                }
                flat_tx = (uint32_t)__popc(__ballot_sync(0xffffffffu, fon)) * (uint32_t)(a.a_bytes / DC_TILE_H) + (uint32_t)a.b_bytes;
            } else {
#pragma unroll
                for (int j = 0; j < MT; ++j) {                      // an absent second tile repeats the first (never stored)
                    const int idx = group * MT + j;
                    const int tile = a.tile_list[idx < n_tiles ? idx : group * MT];
                    const int s = tile / per_stream, t = tile - s * per_stream, ty = t / a.tiles_x, tx = t - ty * a.tiles_x;
                    sN[j] = s; xb[j] = tx * DC_TILE_W * a.sw - a.pw; yb[j] = ty * DC_TILE_H * a.sh - a.ph;
                }
            }
            for (int tap = 0; tap < taps && ok; ++tap) {
                const int ky = tap / a.kw, kx = tap - ky * a.kw;
                for (int cc = 0; cc < a.kchunks && ok; ++cc) {
                    if (lane == 0) {
                        ok = mbar_wait(&ctl->empty[st], ph ^ 1u, ctl, a.status);
                        if (ok && !a.skip_loads) {
                            uint8_t* sa = ring + (size_t)st * stage_bytes;
                            mbar_expect_tx(&ctl->full[st], a.flat ? flat_tx : (uint32_t)stage_bytes);
                            if (!a.flat) {
#pragma unroll
                                for (int j = 0; j < MT; ++j)
                                    tma_load_4d(sa + j * a.a_bytes, &tmA, cc * a.BK, xb[j] + kx, yb[j] + ky, sN[j], &ctl->full[st]);
                            }
                            tma_load_2d(sa + MT * a.a_bytes, &tmB, tap * a.Ci + cc * a.BK, (nb + a.nb_off) * a.BN, &ctl->full[st]);
                        }
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    // the slot is free and its byte count announced (lane 0, above): every lane brings its own group
                    if (a.flat && ok && !a.skip_loads && fon)
                        tma_load_4d(ring + (size_t)st * stage_bytes + (size_t)lane * (a.a_bytes / DC_TILE_H), &tmA, cc * a.BK, fx + kx, fy + ky, fs,
                                    &ctl->full[st]);
                    if (++st == a.stages) { st = 0; ph ^= 1u; }
                }
            }
        }
        // on an abort: give the copies already issued a bounded chance to land before the CTA exits
        if (!ok && lane == 0) {
            const unsigned long long t0 = now_ns();
            while (now_ns() - t0 < 2000000ull) { }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        // Only lane 0 works; descriptors differ from slot to slot in their address bits alone, so the
        // constant upper half is built once and the loop adds (address >> 4).
        if (lane == 0) {
            const uint64_t dconst = umma_desc(0, a.sbo, a.layout_type);
            const uint32_t ring_lo = smem_u32(ring) >> 4, stage_lo = (uint32_t)stage_bytes >> 4, a_lo = (uint32_t)a.a_bytes >> 4;
            const int ksteps = a.BK / 16;
            int st = 0; uint32_t ph = 0, acc = 0, acc_ph = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
                const uint32_t d_tmem = tmem_base + acc * (uint32_t)(MT * a.BN);
                ok = mbar_wait(&ctl->tmem_empty[acc], acc_ph ^ 1u, ctl, a.status);
                tc_fence_after();
                uint32_t accumulate = 0;
                for (int k = 0; k < kiters && ok; ++k) {
                    ok = mbar_wait(&ctl->full[st], ph, ctl, a.status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t adesc0 = dconst + (ring_lo + (uint32_t)st * stage_lo);
                    const uint64_t bdesc = adesc0 + MT * a_lo;
#pragma unroll
                    for (int j = 0; j < MT; ++j) {
                        uint32_t acc_j = accumulate;
                        for (int kk = 0; kk < ksteps; ++kk) {          // 16 bf16 = 32 bytes = 2 descriptor units
                            umma_f16(d_tmem + j * a.BN, adesc0 + j * a_lo + 2 * kk, bdesc + 2 * kk, a.idesc, acc_j);
                            acc_j = 1;
                        }
                    }
                    accumulate = 1;
                    umma_commit(&ctl->empty[st]);                      // frees the slot when these MMAs retire
                    if (++st == a.stages) { st = 0; ph ^= 1u; }
                }
                if (ok) umma_commit(&ctl->tmem_full[acc]);
                if (++acc == (uint32_t)a.nbuf) { acc = 0; acc_ph ^= 1u; }
            }
        }
        __syncwarp();
    } else {
        // ---------------- epilogue ----------------
        epilogue_loop(a, ctl, tmem_base, n_items, n_tiles, warp, lane, blockIdx.x, gridDim.x, a.MT, 0, 0u, a.epi_warps);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(a.tmem_cols) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------
// Few input channels (cin <= 8, e.g. the first layer on RGB): the channels are padded to 8
// (16 bytes per pixel) and the kernel taps are laid side by side along K: K = taps * 8, padded to
// a multiple of 16.  Operands use the unswizzled core-matrix layout.  ONE TMA box per tile brings the
// (16 + kh - 1) x (8 + kw - 1) input patch as pixels of 16 bytes; the rows of tap (ky, kx) are the
// patch pixels starting at (ky * PW + kx), one patch row (PW x 16 bytes) between 8-row groups, so
// every tap is read in place, and one tcgen05.mma (K = 16) consumes two taps whose pixel offsets
// differ by the descriptor's leading-dimension offset.  The packed weights ([K/8][cout][8]) stay
// in shared memory for the whole kernel.  A whole work item is one pipeline stage.
// ---------------------------------------------------------------------------------------------
struct TcSmallArgs {
    TcArgs t;                     // shared fields (BN = cout, NB = 1)
    const __nv_bfloat16* wpacked; // [kblocks][cout][8]
    int kblocks;                  // K / 8 (even); taps = kh * kw real ones, the rest zero
    int w_bytes;                  // kblocks * cout * 16
    int PW, PH, stage_bytes;      // input patch per tile: (8 + kw - 1) x (16 + kh - 1) pixels of 16 bytes, + pad
};

__global__ void __launch_bounds__(kThreadsWide, 1)
k_conv_tc_smallc(const __grid_constant__ CUtensorMap tmA, const TcSmallArgs sa)
{
    extern __shared__ uint8_t smem_raw[];
    const TcArgs& a = sa.t;
    uint8_t* base = (uint8_t*)(((uintptr_t)smem_raw + 127) & ~(uintptr_t)127);
    uint8_t* wsm = base;                                        // packed weights
    uint8_t* ring = wsm + ((sa.w_bytes + 127) & ~127);
    SmemCtl* ctl = (SmemCtl*)(ring + (size_t)a.stages * sa.stage_bytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int per_stream = a.tiles_x * a.tiles_y;
    const int taps = a.kh * a.kw;

    if (threadIdx.x == 0) {
        for (int i = 0; i < a.stages; ++i) { mbar_init(&ctl->full[i], 1); mbar_init(&ctl->empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&ctl->tmem_full[i], 1); mbar_init(&ctl->tmem_empty[i], 32u * (uint32_t)a.epi_warps); }
        ctl->abort_flag = 0;
        ctl->wait_ns = a.wait_ns;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA) : "memory");
    }
    // weights into shared memory; zero the ring once: each slot ends in a pad that no TMA box fills but
    // the last (zero-weight) K block reads, and 0 x garbage could be NaN
    for (int i = threadIdx.x; i < sa.w_bytes / 16; i += blockDim.x)
        ((uint4*)wsm)[i] = __ldg((const uint4*)sa.wpacked + i);
    for (int i = threadIdx.x; i < a.stages * sa.stage_bytes / 16; i += blockDim.x)
        ((uint4*)ring)[i] = make_uint4(0, 0, 0, 0);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> visible to TMA / MMA
    stage_bias(a, ctl, a.epi_warps);
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)), "r"(a.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    pdl_wait();                 // the previous kernel's output, the tile list and its count are read from here on
    pdl_release();
    const int n_items = *a.tile_count;

    if (warp == 0) {
        if (lane == 0) {                                        // producer: one patch per item
            int st = 0; uint32_t ph = 0;
            bool ok = true;
            int tile_next = a.tile_list[blockIdx.x];            // fetched one item ahead: off the critical path
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
                const int tile = tile_next;
                if (item + (int)gridDim.x < n_items) tile_next = a.tile_list[item + gridDim.x];
                const int s = tile / per_stream, t = tile - s * per_stream, ty = t / a.tiles_x, tx = t - ty * a.tiles_x;
                ok = mbar_wait(&ctl->empty[st], ph ^ 1u, ctl, a.status);
                if (!ok) break;
                if (!a.skip_loads) {
                    mbar_expect_tx(&ctl->full[st], (uint32_t)(sa.PW * sa.PH * 16));
                    tma_load_4d(ring + (size_t)st * sa.stage_bytes, &tmA, 0, tx * DC_TILE_W - a.pw, ty * DC_TILE_H - a.ph, s, &ctl->full[st]);
                }
                if (++st == a.stages) { st = 0; ph ^= 1u; }
            }
            if (!ok) { const unsigned long long t0 = now_ns(); while (now_ns() - t0 < 2000000ull) { } }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {                                        // MMA issuer
            const uint32_t b_lbo = (uint32_t)a.Co * 16u;
            const uint64_t bconst = umma_desc(smem_u32(wsm), 128, 0, b_lbo);
            const uint32_t ring_lo = smem_u32(ring) >> 4, stage_lo = (uint32_t)sa.stage_bytes >> 4;
            const uint64_t hi = umma_desc(0, (uint32_t)sa.PW * 16u, 0, 0);     // SBO = one patch row; LBO added per K step
            int st = 0; uint32_t ph = 0, acc = 0, acc_ph = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
                ok = mbar_wait(&ctl->tmem_empty[acc], acc_ph ^ 1u, ctl, a.status);
                if (ok) ok = mbar_wait(&ctl->full[st], ph, ctl, a.status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * (uint32_t)a.BN;
                const uint32_t patch_lo = ring_lo + (uint32_t)st * stage_lo;
                // K step kk covers taps 2kk and 2kk+1: two 16-byte pixel columns of the patch, `lbo` apart
                int tap = 0, ky = 0, kx = 0;
                for (int kk = 0; kk < sa.kblocks / 2; ++kk) {
                    const uint32_t off0 = (uint32_t)(ky * sa.PW + kx);
                    if (++kx == a.kw) { kx = 0; ++ky; }
                    ++tap;
                    uint32_t off1 = off0 + 1;                      // past the last tap: any finite data (its weights are zero)
                    if (tap < taps) { off1 = (uint32_t)(ky * sa.PW + kx); if (++kx == a.kw) { kx = 0; ++ky; } }
                    ++tap;
                    const uint64_t adesc = hi + (patch_lo + off0) + ((uint64_t)(off1 - off0) << 16);
                    umma_f16(d_tmem, adesc, bconst + (uint64_t)(kk * ((2 * b_lbo) >> 4)), a.idesc, kk != 0);
                }
                umma_commit(&ctl->empty[st]);
                umma_commit(&ctl->tmem_full[acc]);
                if (++st == a.stages) { st = 0; ph ^= 1u; }
                if (++acc == 2u) { acc = 0; acc_ph ^= 1u; }
            }
        }
        __syncwarp();
    } else {
        epilogue_loop(a, ctl, tmem_base, n_items, n_items, warp, lane, blockIdx.x, gridDim.x, 1, 0, 0u, a.epi_warps);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(a.tmem_cols) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------
// Input-patch reuse ("halo") variant for stride-1 k x k convolutions with cin a multiple of 64.
// k_conv_tc fetches the 16x8 input window once per kernel tap (9 x 16 KB for 3x3); here the
// (16 + kh - 1) x (8 + kw - 1) patch is fetched ONCE per 64-channel chunk and every tap reads it
// in place.  That needs an operand layout whose rows may start at any patch pixel: the
// unswizzled core-matrix layout with the patch stored as 8 planes (one per 8 channels = 16
// bytes) of [patch row][patch column] pixels.  A tile is 8 pixels wide, so the 8 rows of one
// operand group are the 8 consecutive pixels of one image row, and groups are one patch row
// (PW x 16 bytes) apart: SBO = PW * 16, LBO = plane size, start = plane + (ky * PW + kx) * 16.
// Weights are pre-packed per (channel block, tap, chunk) as [k/8][BN][8] and arrive with one
// plain bulk copy each.
// ---------------------------------------------------------------------------------------------
struct TcHaloArgs {
    TcArgs t;
    const __nv_bfloat16* wpacked;    // [NB][taps][kchunks][8][BN][8]
    int PW, PH, plane_bytes, patch_bytes, a_stages;
};

__device__ __forceinline__ void bulk_copy_g2s(void* dst, const void* src, uint32_t bytes, void* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// SLAB = false: the A side of a 64-channel chunk is one (16 + kh - 1) x (8 + kw - 1) patch in eight 16-byte planes
//               (unswizzled core matrices), read in place by every tap.
// SLAB = true:  the A side of a (chunk, kx) pair is one column slab: the (16 + kh - 1) x 8 pixels of the tile's
//               columns displaced by kx, 128 bytes (64 channels) per pixel, 128-byte swizzled.  The eight pixels of
//               a tile row are one 1024-byte swizzle atom, so tap (ky, kx) is the slab from atom ky on: a plain
//               K-major tile.  kw loads of whole 128-byte rows per chunk instead of kh * kw (tap by tap) or eight
//               loads of 16-byte rows (patch).  ha.patch_bytes then holds the bytes of one slab.
template <int MT, bool SLAB>
__global__ void __launch_bounds__(kThreadsWide, 1)
k_conv_tc_halo(const __grid_constant__ CUtensorMap tmA, const TcHaloArgs ha)
{
    extern __shared__ uint8_t smem_raw[];
    const TcArgs& a = ha.t;
    constexpr uintptr_t kAlign = SLAB ? 1023 : 127;           // swizzle atoms start on 1024-byte boundaries
    uint8_t* aring = (uint8_t*)(((uintptr_t)smem_raw + kAlign) & ~kAlign);
    const int a_slot = MT * ha.patch_bytes;
    uint8_t* bring = aring + (size_t)ha.a_stages * a_slot;
    SmemCtl* ctl = (SmemCtl*)(bring + (size_t)a.stages * a.b_bytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int per_stream = a.tiles_x * a.tiles_y;
    const int taps = a.kh * a.kw;

    if (threadIdx.x == 0) {
        for (int i = 0; i < a.stages; ++i) { mbar_init(&ctl->full[i], 1); mbar_init(&ctl->empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&ctl->tmem_full[i], 1); mbar_init(&ctl->tmem_empty[i], 32u * (uint32_t)a.epi_warps); }
        for (int i = 0; i < 4; ++i) { mbar_init(&ctl->a_full[i], 1); mbar_init(&ctl->a_empty[i], 1); }
        ctl->abort_flag = 0;
        ctl->wait_ns = a.wait_ns;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA) : "memory");
    }
    stage_bias(a, ctl, a.epi_warps);
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)), "r"(a.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    pdl_wait();                 // the previous kernel's output, the tile list and its count are read from here on
    pdl_release();
    const int n_tiles = *a.tile_count;
    const int n_items = (n_tiles + MT - 1) / MT * a.NB;

    if (warp == 0) {
        // ---------------- producer: patches by TMA, weights by bulk copy ----------------
        int sa = 0, sb = 0; uint32_t pa = 0, pb = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
            const int group = item / a.NB, nb = item % a.NB;
            int sN[MT], xb[MT], yb[MT];
#pragma unroll
            for (int j = 0; j < MT; ++j) {
                const int idx = group * MT + j;
                const int tile = a.tile_list[idx < n_tiles ? idx : group * MT];
                const int s = tile / per_stream, t = tile - s * per_stream, ty = t / a.tiles_x, tx = t - ty * a.tiles_x;
                sN[j] = s; xb[j] = tx * DC_TILE_W - a.pw; yb[j] = ty * DC_TILE_H - a.ph;
            }
            for (int cc = 0; cc < a.kchunks && ok; ++cc) {
                for (int kx = 0; kx < (SLAB ? a.kw : 1) && ok; ++kx) {
                    if (lane == 0) {
                        ok = mbar_wait(&ctl->a_empty[sa], pa ^ 1u, ctl, a.status);
                        if (ok && !a.skip_loads) {
                            if (SLAB) {
                                mbar_expect_tx(&ctl->a_full[sa], (uint32_t)(MT * ha.patch_bytes));
#pragma unroll
                                for (int j = 0; j < MT; ++j)
                                    tma_load_4d(aring + (size_t)sa * a_slot + j * ha.patch_bytes, &tmA, cc * 64, xb[j] + kx, yb[j], sN[j],
                                                &ctl->a_full[sa]);
                            } else {
                                mbar_expect_tx(&ctl->a_full[sa], (uint32_t)(MT * 8 * ha.PW * ha.PH * 16));
#pragma unroll
                                for (int j = 0; j < MT; ++j)
                                    for (int g = 0; g < 8; ++g)
                                        tma_load_4d(aring + (size_t)sa * a_slot + j * ha.patch_bytes + g * ha.plane_bytes, &tmA,
                                                    cc * 64 + g * 8, xb[j], yb[j], sN[j], &ctl->a_full[sa]);
                            }
                        }
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (++sa == ha.a_stages) { sa = 0; pa ^= 1u; }
                    // the weight tiles that go with this A stage: all taps (patch), or the taps of column kx (slab)
                    for (int t = 0; t < (SLAB ? a.kh : taps) && ok; ++t) {
                        const int tap = SLAB ? t * a.kw + kx : t;
                        if (lane == 0) {
                            ok = mbar_wait(&ctl->empty[sb], pb ^ 1u, ctl, a.status);
                            if (ok && !a.skip_loads) {
                                mbar_expect_tx(&ctl->full[sb], (uint32_t)a.b_bytes);
                                const uint8_t* src = (const uint8_t*)ha.wpacked + ((size_t)((nb + a.nb_off) * taps + tap) * a.kchunks + cc) * a.b_bytes;
                                bulk_copy_g2s(bring + (size_t)sb * a.b_bytes, src, (uint32_t)a.b_bytes, &ctl->full[sb]);
                            }
                        }
                        ok = __shfl_sync(0xffffffffu, ok, 0);
                        if (++sb == a.stages) { sb = 0; pb ^= 1u; }
                    }
                }
            }
        }
        if (!ok && lane == 0) { const unsigned long long t0 = now_ns(); while (now_ns() - t0 < 2000000ull) { } }
    } else if (warp == 1) {
        // ---------------- MMA issuer (lane 0 only) ----------------
        if (lane == 0) {
            const uint32_t b_lbo = (uint32_t)a.BN * 16u;
            // A: patch planes (rows PW * 16 bytes apart, planes along K), or a 128-byte swizzled K-major slab
            const uint64_t aconst = SLAB ? umma_desc(0, 1024, 2) : umma_desc(0, (uint32_t)ha.PW * 16u, 0, (uint32_t)ha.plane_bytes);
            const uint64_t bconst = umma_desc(0, 128, 0, b_lbo);
            const uint32_t aring_lo = smem_u32(aring) >> 4, bring_lo = smem_u32(bring) >> 4;
            const uint32_t a_slot_lo = (uint32_t)a_slot >> 4, patch_lo = (uint32_t)ha.patch_bytes >> 4;
            const uint32_t a_kstep = SLAB ? 2u : (uint32_t)(2 * ha.plane_bytes) >> 4;    // 16 channels further along K
            const uint32_t b_kstep = (2 * b_lbo) >> 4, b_lo = (uint32_t)a.b_bytes >> 4;
            int sa = 0, sb = 0; uint32_t pa = 0, pb = 0, acc = 0, acc_ph = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
                const uint32_t d_tmem = tmem_base + acc * (uint32_t)(MT * a.BN);
                ok = mbar_wait(&ctl->tmem_empty[acc], acc_ph ^ 1u, ctl, a.status);
                tc_fence_after();
                uint32_t accumulate = 0;
                for (int cc = 0; cc < a.kchunks && ok; ++cc) {
                    for (int ax = 0; ax < (SLAB ? a.kw : 1) && ok; ++ax) {     // A stages of this chunk: one patch, or kw slabs
                        ok = mbar_wait(&ctl->a_full[sa], pa, ctl, a.status);
                        const uint64_t apatch = aconst + (aring_lo + (uint32_t)sa * a_slot_lo);
                        // patch: taps in (ky, kx) order at (ky * PW + kx) * 16 bytes; slab ax: taps (ky, ax) at ky atoms of 1024 bytes
                        const int n_t = SLAB ? a.kh : taps;
                        for (int t = 0; t < n_t && ok; ++t) {
                            const uint32_t tap_lo = SLAB ? (uint32_t)t * 64u : (uint32_t)((t / a.kw) * ha.PW + t % a.kw);
                            ok = mbar_wait(&ctl->full[sb], pb, ctl, a.status);
                            if (!ok) break;
                            tc_fence_after();
                            const uint64_t bdesc = bconst + (bring_lo + (uint32_t)sb * b_lo);
#pragma unroll
                            for (int j = 0; j < MT; ++j) {
                                const uint64_t adesc = apatch + j * patch_lo + tap_lo;
                                uint32_t acc_j = accumulate;
#pragma unroll
                                for (int kk = 0; kk < 4; ++kk) {        // K = 16 per instruction, 64 channels per chunk
                                    umma_f16(d_tmem + j * a.BN, adesc + kk * a_kstep, bdesc + kk * b_kstep, a.idesc, acc_j);
                                    acc_j = 1;
                                }
                            }
                            accumulate = 1;
                            umma_commit(&ctl->empty[sb]);
                            if (++sb == a.stages) { sb = 0; pb ^= 1u; }
                        }
                        if (ok) umma_commit(&ctl->a_empty[sa]);         // the A stage is free once its taps retire
                        if (++sa == ha.a_stages) { sa = 0; pa ^= 1u; }
                    }
                }
                if (ok) umma_commit(&ctl->tmem_full[acc]);
                if (++acc == (uint32_t)a.nbuf) { acc = 0; acc_ph ^= 1u; }
            }
        }
        __syncwarp();
    } else {
        epilogue_loop(a, ctl, tmem_base, n_items, n_tiles, warp, lane, blockIdx.x, gridDim.x, a.MT, 0, 0u, a.epi_warps);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(a.tmem_cols) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------
// CTA pairs (tcgen05.mma.cta_group::2): the column-slab scheme with one 256-row tile pair per work item.
// Wide layers are bound by their weights: per 64-channel chunk a tile needs 54 KB of input slabs but 288 KB of
// weights at 256 output channels.  Here the two CTAs of a cluster (two SMs of one TPC) take one tile each and HALF of
// the item's output channels' weights each; one MMA instruction, issued by the leader (rank 0), reads both CTAs'
// operands (M = 256: 128 rows from each CTA's slab; N = BN: BN / 2 columns from each CTA's weight tile) and
// accumulates into both CTAs' tensor memory (each holds its own tile's 128 rows x BN columns).  Per tile the weight
// traffic into an SM halves, and the accumulators stay double buffered (2 x BN <= 512 columns per CTA).
//
// Every load is a plain per-CTA TMA load into the CTA's own shared memory (no multicast anywhere); the loads of the
// second CTA report their bytes to the leader's barrier (cta_group::2 form of the load), because the leader's MMA
// thread is the only consumer.  Barriers: full / a_full / tmem_empty live in the leader and collect both CTAs;
// empty / a_empty / tmem_full exist in each CTA and are signalled in both by the leader's tcgen05.commit.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_cta(const void* p, uint32_t rank)      // shared::cluster address of p in CTA `rank`
{
    uint32_t out;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(out) : "r"(smem_u32(p)), "r"(rank));
    return out;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// loads into this CTA's shared memory whose bytes are counted on the barrier at shared::cluster address `bar` (the leader's)
__device__ __forceinline__ void tma_load_4d_pair(void* dst, const CUtensorMap* tm, int c0, int c1, int c2, int c3, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
                 ::"r"(smem_u32(dst)), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(void* dst, const CUtensorMap* tm, int c0, int c1, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(smem_u32(dst)), "l"(tm), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void umma_f16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// arrives, once the MMAs issued so far have retired, on the barrier at this offset in both CTAs of the pair
__device__ __forceinline__ void umma_commit_pair(void* bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"((uint16_t)3) : "memory");
}

// ha.t.BN: output channels per item (both CTAs together); ha.t.b_bytes: one CTA's weight tile (BN / 2 rows of 128 bytes);
// tmW: the packed weights [2 NB][taps][kchunks][8][BN / 2][8] seen as rows of 128 bytes.
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
k_conv_tc_pair(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW, const TcHaloArgs ha)
{
    extern __shared__ uint8_t smem_raw[];
    const TcArgs& a = ha.t;
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const uint32_t rank = cluster_rank();
    const bool leader = rank == 0;
    uint8_t* aring = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int a_slot = ha.patch_bytes;                        // one slab
    uint8_t* bring = aring + (size_t)ha.a_stages * a_slot;
    SmemCtl* ctl = (SmemCtl*)(bring + (size_t)a.stages * a.b_bytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int per_stream = a.tiles_x * a.tiles_y;
    const int taps = a.kh * a.kw;

    if (threadIdx.x == 0) {
        for (int i = 0; i < a.stages; ++i) { mbar_init(&ctl->full[i], 1); mbar_init(&ctl->empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&ctl->tmem_full[i], 1); mbar_init(&ctl->tmem_empty[i], 256); }
        for (int i = 0; i < 4; ++i) { mbar_init(&ctl->a_full[i], 1); mbar_init(&ctl->a_empty[i], 1); }
        ctl->abort_flag = 0;
        ctl->wait_ns = a.wait_ns;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmW) : "memory");
    }
    stage_bias(a, ctl, 4);
    if (warp == 1) {                                          // the same warp in both CTAs: tensor memory of the pair
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)), "r"(a.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                       // both CTAs' barriers exist before either is signalled from outside
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    pdl_wait();                 // the previous kernel's output, the tile list and its count are read from here on
    pdl_release();
    const int n_tiles = *a.tile_count;
    const int n_items = (n_tiles + 1) / 2 * a.NB;

    if (warp == 0) {
        // ---------------- producer: this CTA's slab and its half of the weights ----------------
        const uint32_t a_full0 = map_to_cta(&ctl->a_full[0], 0), full0 = map_to_cta(&ctl->full[0], 0);   // the leader's barriers
        int sa = 0, sb = 0; uint32_t pa = 0, pb = 0;
        bool ok = true;
        const int rows_per_tile = a.b_bytes >> 7;             // weight rows of 128 bytes in one CTA's tile
        for (int item = pair; item < n_items && ok; item += n_pairs) {
            const int group = item / a.NB, nb = item % a.NB;
            const int idx = group * 2 + (int)rank;
            const int tile = a.tile_list[idx < n_tiles ? idx : group * 2];      // an absent second tile repeats the first (never stored)
            const int s = tile / per_stream, t = tile - s * per_stream, ty = t / a.tiles_x, tx = t - ty * a.tiles_x;
            const int xb = tx * DC_TILE_W - a.pw, yb = ty * DC_TILE_H - a.ph;
            for (int cc = 0; cc < a.kchunks && ok; ++cc) {
                for (int kx = 0; kx < a.kw && ok; ++kx) {
                    if (lane == 0) {
                        ok = mbar_wait(&ctl->a_empty[sa], pa ^ 1u, ctl, a.status);
                        if (ok && !a.skip_loads) {
                            if (leader) mbar_expect_tx(&ctl->a_full[sa], (uint32_t)(2 * ha.patch_bytes));
                            tma_load_4d_pair(aring + (size_t)sa * a_slot, &tmA, cc * 64, xb + kx, yb, s, a_full0 + (uint32_t)sa * 8u);
                        }
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (++sa == ha.a_stages) { sa = 0; pa ^= 1u; }
                    for (int t2 = 0; t2 < a.kh && ok; ++t2) {
                        const int tap = t2 * a.kw + kx;
                        if (lane == 0) {
                            ok = mbar_wait(&ctl->empty[sb], pb ^ 1u, ctl, a.status);
                            if (ok && !a.skip_loads) {
                                if (leader) mbar_expect_tx(&ctl->full[sb], (uint32_t)(2 * a.b_bytes));
                                const int row = (((nb * 2 + (int)rank) * taps + tap) * a.kchunks + cc) * rows_per_tile;
                                tma_load_2d_pair(bring + (size_t)sb * a.b_bytes, &tmW, 0, row, full0 + (uint32_t)sb * 8u);
                            }
                        }
                        ok = __shfl_sync(0xffffffffu, ok, 0);
                        if (++sb == a.stages) { sb = 0; pb ^= 1u; }
                    }
                }
            }
        }
        if (!ok && lane == 0) { const unsigned long long t0 = now_ns(); while (now_ns() - t0 < 2000000ull) { } }
    } else if (warp == 1) {
        // ---------------- MMA issuer: the leader's lane 0 issues for both CTAs ----------------
        if (leader && lane == 0) {
            const uint32_t b_lbo = (uint32_t)(a.BN / 2) * 16u;
            const uint64_t aconst = umma_desc(0, 1024, 2);
            const uint64_t bconst = umma_desc(0, 128, 0, b_lbo);
            const uint32_t aring_lo = smem_u32(aring) >> 4, bring_lo = smem_u32(bring) >> 4;
            const uint32_t a_slot_lo = (uint32_t)a_slot >> 4;
            const uint32_t b_kstep = (2 * b_lbo) >> 4, b_lo = (uint32_t)a.b_bytes >> 4;
            int sa = 0, sb = 0; uint32_t pa = 0, pb = 0, acc = 0, acc_ph = 0;
            bool ok = true;
            for (int item = pair; item < n_items && ok; item += n_pairs) {
                const uint32_t d_tmem = tmem_base + acc * (uint32_t)a.BN;
                ok = mbar_wait(&ctl->tmem_empty[acc], acc_ph ^ 1u, ctl, a.status);
                tc_fence_after();
                uint32_t accumulate = 0;
                for (int cc = 0; cc < a.kchunks && ok; ++cc) {
                    for (int ax = 0; ax < a.kw && ok; ++ax) {
                        ok = mbar_wait(&ctl->a_full[sa], pa, ctl, a.status);
                        const uint64_t aslab = aconst + (aring_lo + (uint32_t)sa * a_slot_lo);
                        for (int t = 0; t < a.kh && ok; ++t) {               // tap (t, ax): the slab from swizzle atom t on
                            ok = mbar_wait(&ctl->full[sb], pb, ctl, a.status);
                            if (!ok) break;
                            tc_fence_after();
                            const uint64_t bdesc = bconst + (bring_lo + (uint32_t)sb * b_lo);
                            const uint64_t adesc = aslab + (uint32_t)t * 64u;
#pragma unroll
                            for (int kk = 0; kk < 4; ++kk) {                 // K = 16 per instruction, 64 channels per chunk
                                umma_f16_pair(d_tmem, adesc + kk * 2u, bdesc + kk * b_kstep, a.idesc, accumulate);
                                accumulate = 1;
                            }
                            umma_commit_pair(&ctl->empty[sb]);
                            if (++sb == a.stages) { sb = 0; pb ^= 1u; }
                        }
                        if (ok) umma_commit_pair(&ctl->a_empty[sa]);
                        if (++sa == ha.a_stages) { sa = 0; pa ^= 1u; }
                    }
                }
                if (ok) umma_commit_pair(&ctl->tmem_full[acc]);
                if (++acc == 2u) { acc = 0; acc_ph ^= 1u; }
            }
        }
        __syncwarp();
    } else {
        // ---------------- epilogue: this CTA's tile; the accumulator is handed back on the leader's barrier ----------------
        const uint32_t remote_empty = map_to_cta(&ctl->tmem_empty[0], 0);
        epilogue_loop(a, ctl, tmem_base, n_items, n_tiles, warp, lane, pair, n_pairs, 2, (int)rank, remote_empty);
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                       // neither CTA frees tensor memory or leaves while the other may still use it
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(a.tmem_cols) : "memory");
    }
}

// weights [cout][taps][cin] -> [NB][taps][kchunks][8][BN][8]
__global__ void k_pack_halo(const __nv_bfloat16* w, int cout, int taps, int cin, int BN, __nv_bfloat16* out)
{
    const int kchunks = cin / 64;
    const size_t total = (size_t)cout * taps * cin;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        size_t r = i;
        const int e = (int)(r & 7); r >>= 3;
        const int n = (int)(r % BN); r /= BN;
        const int k8 = (int)(r & 7); r >>= 3;
        const int cc = (int)(r % kchunks); r /= kchunks;
        const int tap = (int)(r % taps); const int nb = (int)(r / taps);
        out[i] = w[((size_t)(nb * BN + n) * taps + tap) * cin + cc * 64 + k8 * 8 + e];
    }
}

// [S][H][W][C] -> [S][H][W][8] with zero padding, C <= 8
__global__ void k_pad_channels8(const __nv_bfloat16* in, size_t pixels, int C, __nv_bfloat16* out)
{
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < pixels; i += (size_t)gridDim.x * blockDim.x) {
        unsigned short v[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        const unsigned short* p = (const unsigned short*)in + i * C;
        for (int c = 0; c < C; ++c) v[c] = p[c];
        ((uint4*)out)[i] = make_uint4(v[0] | ((uint32_t)v[1] << 16), v[2] | ((uint32_t)v[3] << 16),
                                      v[4] | ((uint32_t)v[5] << 16), v[6] | ((uint32_t)v[7] << 16));
    }
}

// [S][H][W][C] -> [S][H][W][16] with zero padding, C < 16
__global__ void k_pad_channels16(const __nv_bfloat16* in, size_t pixels, int C, __nv_bfloat16* out)
{
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < pixels; i += (size_t)gridDim.x * blockDim.x) {
        unsigned short v[16];
#pragma unroll
        for (int c = 0; c < 16; ++c) v[c] = 0;
        const unsigned short* p = (const unsigned short*)in + i * C;
        for (int c = 0; c < C; ++c) v[c] = p[c];
        ((uint4*)out)[2 * i] = make_uint4(v[0] | ((uint32_t)v[1] << 16), v[2] | ((uint32_t)v[3] << 16),
                                          v[4] | ((uint32_t)v[5] << 16), v[6] | ((uint32_t)v[7] << 16));
        ((uint4*)out)[2 * i + 1] = make_uint4(v[8] | ((uint32_t)v[9] << 16), v[10] | ((uint32_t)v[11] << 16),
                                              v[12] | ((uint32_t)v[13] << 16), v[14] | ((uint32_t)v[15] << 16));
    }
}

// weights [cout][taps][cin] -> [cout][taps][16], channels beyond cin zero
__global__ void k_pack_pad16(const __nv_bfloat16* w, size_t cout_taps, int cin, __nv_bfloat16* out)
{
    const size_t total = cout_taps * 16;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const size_t ct = i >> 4; const int ch = (int)(i & 15);
        out[i] = ch < cin ? w[ct * cin + ch] : __float2bfloat16(0.f);
    }
}

// weights [cout][taps][cin] -> [kblocks][cout][8]: block j holds tap j (cin real channels, rest zero)
__global__ void k_pack_smallc(const __nv_bfloat16* w, int cout, int taps, int cin, int kblocks, __nv_bfloat16* out)
{
    const int total = kblocks * cout * 8;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
        const int e = i & 7, n = (i >> 3) % cout, j = (i >> 3) / cout;
        out[i] = (j < taps && e < cin) ? w[((size_t)n * taps + j) * cin + e] : __float2bfloat16_rn(0.f);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
        cudaGetLastError();
    }
    return fn;
}

// Tensor maps are encoded once per (base address, operand scheme, channel block) and kept with the layer: in steady
// state a launch finds its maps in these slots.  A new base or scheme (the tuner's trials, a caller's own buffers in
// dc_conv_partial) replaces a slot.
static_assert(sizeof(CUtensorMap) == 128, "dc_tm_slot stores a CUtensorMap");
static CUtensorMap* tm_find(dc_tm_slot* slots, int n, int* next, const void* base, int code, int bn, bool* hit)
{
    for (int i = 0; i < n; ++i)
        if (slots[i].valid && slots[i].base == base && slots[i].code == code && slots[i].bn == bn) {
            *hit = true;
            return (CUtensorMap*)slots[i].map;
        }
    int k = 0;
    if (n > 1) { k = *next % n; *next = (k + 1) % n; }
    slots[k].valid = true; slots[k].base = base; slots[k].code = code; slots[k].bn = bn;
    *hit = false;
    return (CUtensorMap*)slots[k].map;
}
static void tm_drop(dc_tm_slot* slots, int n, const CUtensorMap* m)
{
    for (int i = 0; i < n; ++i) if ((const CUtensorMap*)slots[i].map == m) slots[i].valid = false;
}

// Two CTAs may share an SM when each needs at most 256 TMEM columns; each then gets half the operand-ring budget.
// Layers with few output channels or a short K are bound by the epilogue (TMEM -> registers -> global), and a
// second resident CTA doubles the epilogue warps per SM.
static uint32_t tmem_cols_for(int nbuf, int mt, int bn)
{
    uint32_t need = (uint32_t)(nbuf * mt * bn), cols = 32;
    while (cols < need) cols <<= 1;
    return cols;
}
// Operand-ring bytes of a CTA that has its SM alone: 200 KB, or 182 KB while the cache's matcher runs beside the
// inference (dc_lookahead_frame): with 182 KB a convolution CTA leaves room for one CTA of the block search (32 KB) on
// its SM, which then works in the tensor-core kernel's idle issue slots instead of waiting for a free SM.  Set per
// launch from the cache's state.
// Launch with programmatic stream serialization allowed (see pdl_wait): the kernel may start before the previous
// kernel of the stream has ended.  Not while the block search of the next frame runs beside the inference: there the
// search is the longer chain, and it is the gaps between convolution kernels that let more of its CTAs in.
// DC_NO_PDL=1 (diagnostics) always launches the ordinary way.
static thread_local bool t_pdl = true;
template <typename... KArgs, typename... Args>
static cudaError_t launch_conv_kernel(void (*kernel)(KArgs...), int grid, int threads, size_t smem, cudaStream_t stream, Args&&... args)
{
    static const bool pdl_env = getenv("DC_NO_PDL") == nullptr;
    const bool pdl = pdl_env && t_pdl;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3((unsigned)threads); cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

static thread_local int t_ring_kb = 200;
static thread_local int t_epi_warps = 4;      // the layer's tuned epilogue width, honoured by launches with one CTA per SM
static int epi_warps_for(int ctas) { return t_epi_warps == 8 && ctas != 2 ? 8 : 4; }
static thread_local int t_bias_bytes = 0;     // the launch's bias values staged in shared memory (0: too many, read from global memory)
static int bias_bytes_for(const dc_layer_desc& group) { return group.cout * 4 <= 16384 ? (group.cout * 4 + 15) & ~15 : 0; }
// eight epilogue warps stage twice as much, and every CTA keeps its bias values: the rings give that up
static int ring_budget(int ctas)
{
    const int n = ctas == 2 ? 2 : 1;
    return (t_ring_kb * 1024 - (epi_warps_for(ctas) == 8 ? 4 * kStageBytes : 0) - n * t_bias_bytes) / n;
}

// Every launch waits at most kWaitLimitNs on the device.  dc_debug_stall_next_conv (below) arms the next launch
// only: its producer issues no copy and its waits run out after the given time.
static void set_wait_limit(dc_cache* c, TcArgs& a)
{
    a.wait_ns = kWaitLimitNs; a.skip_loads = 0;
    if (c->debug_stall_ms > 0) {
        a.wait_ns = (unsigned long long)c->debug_stall_ms * 1000000ull;
        a.skip_loads = 1;
        c->debug_stall_ms = 0;
    }
}

// A grouped convolution (AlexNet's layers 2, 4, 5) is `groups` independent convolutions, each from its own slice of
// the input channels to its own slice of the output channels.  One launch per group: the input tensor map starts at
// the group's first channel and spans the group's channels only (pixels keep the full layer's pitch), the weights
// [cout][kh][kw][cin / groups] need no slicing, and the kernel adds the group's first channel block (nb_off) to the
// channel blocks it reads weights for and writes.  This is the layer as one group sees it.
static int n_groups(const dc_layer_desc& d) { return d.groups > 1 ? d.groups : 1; }
static dc_layer_desc group_view(const dc_layer_desc& d)
{
    dc_layer_desc g = d;
    g.cin = d.cin / n_groups(d); g.cout = d.cout / n_groups(d); g.groups = 1;
    return g;
}

struct TcPlan { int BK, BN, NB, MT, nbuf, stages, a_bytes, b_bytes; CUtensorMapSwizzle swz; uint32_t layout_type, sbo; size_t smem; };

bool make_plan(const dc_layer_desc& d, TcPlan& p, int want_mt = 0, int want_bn = 0, int ctas = 1)
{
    if (d.kind != DC_CONV) return false;
    if (d.sh < 1 || d.sw < 1 || DC_TILE_W * d.sw > 256 || DC_TILE_H * d.sh > 256) return false;   // TMA box limit
    if (d.cin % 64 == 0) { p.BK = 64; p.swz = CU_TENSOR_MAP_SWIZZLE_128B; p.layout_type = 2; }
    else if (d.cin % 32 == 0) { p.BK = 32; p.swz = CU_TENSOR_MAP_SWIZZLE_64B; p.layout_type = 4; }
    else if (d.cin % 16 == 0) { p.BK = 16; p.swz = CU_TENSOR_MAP_SWIZZLE_32B; p.layout_type = 6; }
    else return false;
    p.BN = 0;
    for (int bn = 256; bn >= 32; bn -= 32) if (d.cout % bn == 0) { p.BN = bn; break; }
    if (!p.BN) return false;
    if (want_bn > 0) {                                           // a tuned choice: must divide cout like the default
        if (want_bn % 32 != 0 || want_bn > 256 || d.cout % want_bn != 0) return false;
        p.BN = want_bn;
    }
    p.NB = d.cout / p.BN;
    p.a_bytes = DC_TILE_PX * p.BK * 2;
    p.b_bytes = p.BN * p.BK * 2;
    p.sbo = 8 * p.BK * 2;
    if (p.b_bytes % 1024 != 0) return false;                    // keep every operand tile on a swizzle-pattern boundary
    // two tiles share each B tile: halves the weight traffic per FLOP; 512 TMEM columns hold
    // MT * BN * nbuf accumulator columns
    p.MT = want_mt > 0 ? want_mt : 1;
    p.nbuf = p.MT * p.BN * 2 <= 512 ? 2 : 1;
    if (ctas == 2 && tmem_cols_for(p.nbuf, p.MT, p.BN) > 256) return false;
    int st = ring_budget(ctas) / (p.MT * p.a_bytes + p.b_bytes);
    p.stages = st > kMaxStages ? kMaxStages : st;
    if (p.stages < 2) return false;
    p.smem = (size_t)p.stages * (p.MT * p.a_bytes + p.b_bytes) + ctl_bytes(epi_warps_for(ctas)) + t_bias_bytes + 1024;
    return true;
}

struct HaloPlan { int BN, NB, PW, PH, plane_bytes, patch_bytes, b_bytes; };

bool halo_ok(const dc_layer_desc& d, HaloPlan& h, int want_bn = 0)
{
    if (d.kind != DC_CONV || d.sh != 1 || d.sw != 1 || d.cin % 64 != 0 || d.kh * d.kw < 2 || d.kh > 5 || d.kw > 5) return false;
    h.BN = 0;
    for (int bn = 256; bn >= 32; bn -= 32) if (d.cout % bn == 0) { h.BN = bn; break; }
    if (!h.BN) return false;
    if (want_bn > 0) {                                           // a tuned choice: must divide cout like the default
        if (want_bn % 32 != 0 || want_bn > 256 || d.cout % want_bn != 0) return false;
        h.BN = want_bn;
    }
    h.NB = d.cout / h.BN;
    h.PW = DC_TILE_W + d.kw - 1; h.PH = DC_TILE_H + d.kh - 1;
    h.plane_bytes = (h.PW * h.PH * 16 + 127) & ~127;       // TMA destinations are 128-byte aligned
    h.patch_bytes = 8 * h.plane_bytes;
    h.b_bytes = h.BN * 128;
    return true;
}

bool smallc_ok(const dc_layer_desc& d)
{
    return d.kind == DC_CONV && d.sh == 1 && d.sw == 1 && d.cin <= 8 && d.cout % 32 == 0 && d.cout <= 256 &&
           d.kh * d.kw <= 64;
}

// Few input channels with a stride or a large kernel (e.g. 11 x 11 stride 4 on RGB): the channels are padded
// to 16 and the layer runs on the tap-by-tap kernel as a 16-channel convolution (K = taps x 16; the padded
// products are zeros).  Far more tensor work than needed, still many times faster than the CUDA-core kernel.
dc_layer_desc padded16(const dc_layer_desc& d) { dc_layer_desc e = d; e.cin = 16; return e; }
bool pad16_ok(const dc_layer_desc& d)
{
    TcPlan p;
    return d.kind == DC_CONV && d.cin < 16 && !make_plan(d, p) && !smallc_ok(d) && make_plan(padded16(d), p);
}

}  // namespace

int dc_conv_bf16_supported(const dc_cache* c, int layer)
{
    TcPlan p;
    if (getenv("DC_NO_TENSOR_CORES")) return 0;
    if (c->cfg.dtype != DC_BF16 || encode_fn() == nullptr) return 0;
    if (n_groups(c->L[layer].d) > 1) {                            // per group: the tap-by-tap kernel or the patch / slab kernels
        const dc_layer_desc g = group_view(c->L[layer].d);
        return make_plan(g, p) && (g.cin * 2) % 16 == 0;          // a group's first channel must be 16-byte aligned for its tensor map
    }
    return make_plan(c->L[layer].d, p) || smallc_ok(c->L[layer].d) || pad16_ok(c->L[layer].d);
}

// Normal layers need no repacking ([cout][kh][kw][cin] is already K-major); few-channel layers
// get their tap-major packed copy and a buffer for the channel-padded input.
int dc_pack_weights_bf16(dc_cache* c, int layer)
{
    dc_layer_rt& L = c->L[layer];
    TcPlan p;
    HaloPlan h;
    const dc_layer_desc dg = group_view(L.d);                     // the layer itself when it is not grouped
    if (halo_ok(dg, h)) {
        // [cout][taps][cin / groups]: channel blocks never straddle a group (BN divides cout / groups)
        const size_t n = (size_t)L.d.cout * L.d.kh * L.d.kw * dg.cin;
        DC_CUDA(cudaMalloc(&L.weight_halo, n * 2));
        c->bytes += n * 2;
        int grid = (int)((n + 255) / 256); if (grid > c->num_sms * 8) grid = c->num_sms * 8;
        k_pack_halo<<<grid, 256, 0, c->stream>>>((const __nv_bfloat16*)L.weight, L.d.cout, L.d.kh * L.d.kw, dg.cin, h.BN,
                                                 (__nv_bfloat16*)L.weight_halo);
        L.halo_bn = h.BN;
        DC_CUDA(cudaGetLastError());
    }
    if (n_groups(L.d) > 1) return DC_OK;                          // grouped layers use the kernels above only
    if (pad16_ok(L.d)) {
        const size_t cout_taps = (size_t)L.d.cout * L.d.kh * L.d.kw;
        const size_t wbytes = cout_taps * 16 * 2, pbytes = (size_t)c->S * L.in_h * L.in_w * 32;
        DC_CUDA(cudaMalloc(&L.weight_packed, wbytes));
        DC_CUDA(cudaMalloc(&L.in_padded, pbytes));
        c->bytes += wbytes + pbytes;
        L.k_packed = L.d.kh * L.d.kw * 16;
        k_pack_pad16<<<dc_div_up((int)(cout_taps * 16), 256), 256, 0, c->stream>>>((const __nv_bfloat16*)L.weight, cout_taps, L.d.cin,
                                                                                   (__nv_bfloat16*)L.weight_packed);
        DC_CUDA(cudaGetLastError());
        return DC_OK;
    }
    if (make_plan(L.d, p) || !smallc_ok(L.d)) return DC_OK;
    const int taps = L.d.kh * L.d.kw, kblocks = (taps + 1) / 2 * 2;
    const size_t wbytes = (size_t)kblocks * L.d.cout * 16, pbytes = (size_t)c->S * L.in_h * L.in_w * 16;
    DC_CUDA(cudaMalloc(&L.weight_packed, wbytes));
    DC_CUDA(cudaMalloc(&L.in_padded, pbytes));
    c->bytes += wbytes + pbytes;
    L.k_packed = kblocks * 8;
    k_pack_smallc<<<dc_div_up(kblocks * L.d.cout * 8, 256), 256, 0, c->stream>>>((const __nv_bfloat16*)L.weight, L.d.cout, taps,
                                                                               L.d.cin, kblocks, (__nv_bfloat16*)L.weight_packed);
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}

static int launch_smallc(dc_cache* c, int layer, const void* in, void* out, const int32_t* tile_list,
                         const int32_t* tile_count, const uint32_t* masks, int max_tiles)
{
    dc_layer_rt& L = c->L[layer];
    const dc_layer_desc& d = L.d;
    EncodeTiledFn enc = encode_fn();
    if (!enc || !L.weight_packed) return DC_ERR_CUDA;
    const size_t pixels = (size_t)c->S * L.in_h * L.in_w;
    const int PW = DC_TILE_W + d.kw - 1, PH = DC_TILE_H + d.kh - 1;
    bool hit;
    CUtensorMap* tmAp = tm_find(L.tm_a, 4, &L.tm_next, L.in_padded, 7, 0, &hit);
    if (!hit) {
        cuuint64_t dims[4] = {8, (cuuint64_t)L.in_w, (cuuint64_t)L.in_h, (cuuint64_t)c->S};
        cuuint64_t strides[3] = {16, (cuuint64_t)L.in_w * 16, (cuuint64_t)L.in_h * L.in_w * 16};
        cuuint32_t box[4] = {8, (cuuint32_t)PW, (cuuint32_t)PH, 1};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        if (enc(tmAp, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, L.in_padded, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
            tm_drop(L.tm_a, 4, tmAp);
            return DC_ERR_CUDA;
        }
    }
    const CUtensorMap& tmA = *tmAp;
    TcSmallArgs sa;
    TcArgs& a = sa.t;
    a.bias = L.bias; a.out = (__nv_bfloat16*)out; a.tile_list = tile_list; a.tile_count = tile_count; a.masks = masks;
    a.Ho = d.out_h; a.Wo = d.out_w; a.Co = d.cout; a.Ci = d.cin; a.kh = d.kh; a.kw = d.kw; a.sh = 1; a.sw = 1;
    a.ph = d.ph; a.pw = d.pw; a.relu = d.relu; a.tiles_x = L.tiles_x; a.tiles_y = L.tiles_y;
    a.BN = d.cout; a.NB = 1; a.nb_off = 0; a.MT = 1; a.nbuf = 2; a.BK = 16; a.kchunks = 1; a.a_bytes = 0; a.b_bytes = 0; a.sbo = 128; a.layout_type = 0;
    a.idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(d.cout >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
    a.status = c->status;
    set_wait_limit(c, a);
    sa.wpacked = (const __nv_bfloat16*)L.weight_packed;
    sa.kblocks = L.k_packed / 8;
    sa.w_bytes = sa.kblocks * d.cout * 16;
    sa.PW = PW; sa.PH = PH;
    sa.stage_bytes = (PW * PH * 16 + 128 + 127) & ~127;          // patch + a readable pad behind its last pixel
    const int stage_bytes = sa.stage_bytes;
    const int ctas = L.tc_ctas == 2 && tmem_cols_for(2, 1, d.cout) <= 256 ? 2 : 1;
    a.tmem_cols = tmem_cols_for(2, 1, d.cout);
    int st = (ring_budget(ctas) - sa.w_bytes) / stage_bytes;
    a.stages = st > kMaxStages ? kMaxStages : st;
    if (a.stages < 2) return DC_ERR_CONFIG;
    a.epi_warps = epi_warps_for(ctas);
    a.bias_smem = t_bias_bytes ? d.cout : 0;
    const size_t smem = (size_t)a.stages * stage_bytes + ((sa.w_bytes + 127) & ~127) + ctl_bytes(a.epi_warps) + t_bias_bytes + 256;
    static dc_once_per_device attr_set;
    if (attr_set.first(c->device)) {
        DC_CUDA(cudaFuncSetAttribute(k_conv_tc_smallc, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
    }
    int grid_pad = (int)((pixels + 255) / 256); if (grid_pad > c->num_sms * 8) grid_pad = c->num_sms * 8;
    int items = max_tiles < 1 ? 1 : max_tiles;
    int grid = items > c->num_sms * ctas ? c->num_sms * ctas : items;
    dc_prof_scope ps(c, DC_ST_CONV);
    k_pad_channels8<<<grid_pad, 256, 0, c->stream>>>((const __nv_bfloat16*)in, pixels, d.cin, (__nv_bfloat16*)L.in_padded);
    DC_CUDA(launch_conv_kernel(k_conv_tc_smallc, grid, threads_for(a.epi_warps), smem, c->stream, tmA, sa));
    c->launches += 2;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}

static int launch_halo(dc_cache* c, int layer, int grp, int mt, bool slab, const void* in, void* out, const int32_t* tile_list,
                       const int32_t* tile_count, const uint32_t* masks, int max_tiles)
{
    dc_layer_rt& L = c->L[layer];
    const dc_layer_desc d = group_view(L.d);                      // what one group computes; L.d itself when ungrouped
    const int cin_all = L.d.cin, cout_all = L.d.cout;
    HaloPlan h;
    EncodeTiledFn enc = encode_fn();
    if (!enc || !L.weight_halo || !halo_ok(d, h, L.tc_bn)) return DC_ERR_CONFIG;
    if (L.halo_bn != h.BN) {
        // the packed weights are grouped by channel block: another block width needs another packing (same size).
        // Happens while the tuner tries widths and once more for its final choice, never in steady state.
        const size_t n = (size_t)cout_all * d.kh * d.kw * d.cin;
        int pgrid = (int)((n + 255) / 256); if (pgrid > c->num_sms * 8) pgrid = c->num_sms * 8;
        k_pack_halo<<<pgrid, 256, 0, c->stream>>>((const __nv_bfloat16*)L.weight, cout_all, d.kh * d.kw, d.cin, h.BN,
                                                  (__nv_bfloat16*)L.weight_halo);
        L.halo_bn = h.BN;
    }
    in = (const uint8_t*)in + (size_t)grp * d.cin * 2;            // the group's first input channel
    bool hit;
    CUtensorMap* tmAp = tm_find(L.tm_a, 4, &L.tm_next, in, slab ? 5 : 3, 0, &hit);
    if (!hit) {
        cuuint64_t dims[4] = {(cuuint64_t)d.cin, (cuuint64_t)L.in_w, (cuuint64_t)L.in_h, (cuuint64_t)c->S};
        cuuint64_t strides[3] = {(cuuint64_t)cin_all * 2, (cuuint64_t)L.in_w * cin_all * 2, (cuuint64_t)L.in_h * L.in_w * cin_all * 2};
        cuuint32_t box[4] = {8, (cuuint32_t)h.PW, (cuuint32_t)h.PH, 1};
        if (slab) { box[0] = 64; box[1] = DC_TILE_W; }            // a column slab: 64 channels x 8 pixels x PH rows
        cuuint32_t estr[4] = {1, 1, 1, 1};
        if (enc(tmAp, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(in), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, slab ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
            tm_drop(L.tm_a, 4, tmAp);
            return DC_ERR_CUDA;
        }
    }
    const CUtensorMap& tmA = *tmAp;
    TcHaloArgs ha;
    TcArgs& a = ha.t;
    a.bias = L.bias; a.out = (__nv_bfloat16*)out; a.tile_list = tile_list; a.tile_count = tile_count; a.masks = masks;
    a.Ho = d.out_h; a.Wo = d.out_w; a.Co = cout_all; a.Ci = d.cin; a.kh = d.kh; a.kw = d.kw; a.sh = 1; a.sw = 1;
    a.ph = d.ph; a.pw = d.pw; a.relu = d.relu; a.tiles_x = L.tiles_x; a.tiles_y = L.tiles_y;
    a.BN = h.BN; a.NB = h.NB; a.nb_off = grp * h.NB; a.BK = 64; a.kchunks = d.cin / 64; a.MT = mt; a.nbuf = mt * h.BN * 2 <= 512 ? 2 : 1;
    a.a_bytes = 0; a.b_bytes = h.b_bytes; a.sbo = 128; a.layout_type = 0;
    a.idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(h.BN >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
    a.status = c->status;
    set_wait_limit(c, a);
    ha.wpacked = (const __nv_bfloat16*)L.weight_halo;
    ha.PW = h.PW; ha.PH = h.PH; ha.plane_bytes = h.plane_bytes;
    ha.patch_bytes = slab ? h.PH * DC_TILE_W * 128 : h.patch_bytes;
    // patch ring: as deep as leaves at least 3 weight stages (a small-K item is one patch, so depth = items in flight)
    a.tmem_cols = tmem_cols_for(a.nbuf, mt, h.BN);
    const int ctas = L.tc_ctas == 2 && a.tmem_cols <= 256 ? 2 : 1;
    const int budget = ring_budget(ctas);
    ha.a_stages = 2;
    for (int as = 4; as > 2; --as)
        if (budget - as * mt * ha.patch_bytes >= 3 * h.b_bytes) { ha.a_stages = as; break; }
    const int a_total = ha.a_stages * mt * ha.patch_bytes;
    int st = (budget - a_total) / h.b_bytes;
    a.stages = st > kMaxStages ? kMaxStages : st;
    if (a.stages < 2) return DC_ERR_CONFIG;
    a.epi_warps = epi_warps_for(ctas);
    a.bias_smem = t_bias_bytes ? d.cout : 0;
    const size_t smem = (size_t)a_total + (size_t)a.stages * h.b_bytes + ctl_bytes(a.epi_warps) + t_bias_bytes + (slab ? 1280 : 256);
    if (smem > 227 * 1024) return DC_ERR_CONFIG;
    static dc_once_per_device attr_set;
    if (attr_set.first(c->device)) {
        DC_CUDA(cudaFuncSetAttribute(k_conv_tc_halo<1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        DC_CUDA(cudaFuncSetAttribute(k_conv_tc_halo<2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        DC_CUDA(cudaFuncSetAttribute(k_conv_tc_halo<1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        DC_CUDA(cudaFuncSetAttribute(k_conv_tc_halo<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
    }
    long long items = (long long)(((max_tiles < 1 ? 1 : max_tiles) + mt - 1) / mt) * h.NB;
    int grid = items > c->num_sms * ctas ? c->num_sms * ctas : (int)items;
    dc_prof_scope ps(c, DC_ST_CONV);
    if (slab) {
        if (mt == 2) DC_CUDA(launch_conv_kernel(k_conv_tc_halo<2, true>, grid, threads_for(a.epi_warps), smem, c->stream, tmA, ha));
        else DC_CUDA(launch_conv_kernel(k_conv_tc_halo<1, true>, grid, threads_for(a.epi_warps), smem, c->stream, tmA, ha));
    } else {
        if (mt == 2) DC_CUDA(launch_conv_kernel(k_conv_tc_halo<2, false>, grid, threads_for(a.epi_warps), smem, c->stream, tmA, ha));
        else DC_CUDA(launch_conv_kernel(k_conv_tc_halo<1, false>, grid, threads_for(a.epi_warps), smem, c->stream, tmA, ha));
    }
    c->launches += 1;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}

// The CTA-pair kernel takes stride-1 layers with cin a multiple of 64 (the column-slab conditions) whose output
// channels divide into blocks of 256 or 128 (half a block per CTA).
static bool pair_ok(const dc_layer_desc& d, int& bn)
{
    HaloPlan h;
    if (n_groups(d) > 1 || !halo_ok(d, h)) return false;
    bn = d.cout % 256 == 0 ? 256 : (d.cout % 128 == 0 ? 128 : 0);
    return bn != 0;
}

static int launch_pair(dc_cache* c, int layer, const void* in, void* out, const int32_t* tile_list,
                       const int32_t* tile_count, const uint32_t* masks, int max_tiles)
{
    dc_layer_rt& L = c->L[layer];
    const dc_layer_desc& d = L.d;
    EncodeTiledFn enc = encode_fn();
    int bn = 0;
    if (!enc || !L.weight_halo || !pair_ok(d, bn)) return DC_ERR_CONFIG;
    const int half = bn / 2, taps = d.kh * d.kw, kchunks = d.cin / 64;
    if (L.halo_bn != half) {                                     // weights grouped by half blocks: [2 NB][taps][kchunks][8][half][8]
        const size_t n = (size_t)d.cout * taps * d.cin;
        int pgrid = (int)((n + 255) / 256); if (pgrid > c->num_sms * 8) pgrid = c->num_sms * 8;
        k_pack_halo<<<pgrid, 256, 0, c->stream>>>((const __nv_bfloat16*)L.weight, d.cout, taps, d.cin, half, (__nv_bfloat16*)L.weight_halo);
        L.halo_bn = half;
    }
    const int PH = DC_TILE_H + d.kh - 1;
    bool hit_a, hit_b;
    CUtensorMap* tmAp = tm_find(L.tm_a, 4, &L.tm_next, in, 5, 0, &hit_a);     // the column-slab map of the single-CTA kernel
    if (!hit_a) {
        cuuint64_t dims[4] = {(cuuint64_t)d.cin, (cuuint64_t)L.in_w, (cuuint64_t)L.in_h, (cuuint64_t)c->S};
        cuuint64_t strides[3] = {(cuuint64_t)d.cin * 2, (cuuint64_t)L.in_w * d.cin * 2, (cuuint64_t)L.in_h * L.in_w * d.cin * 2};
        cuuint32_t box[4] = {64, DC_TILE_W, (cuuint32_t)PH, 1};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        if (enc(tmAp, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(in), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
            tm_drop(L.tm_a, 4, tmAp);
            return DC_ERR_CUDA;
        }
    }
    const int b_bytes = half * 128;                              // one CTA's weight tile: half rows of 64 channels
    CUtensorMap* tmWp = tm_find(&L.tm_b, 1, nullptr, L.weight_halo, 7, half, &hit_b);
    if (!hit_b) {                                                // the packed weights as rows of 128 bytes; a box is one tile
        const cuuint64_t rows = (cuuint64_t)d.cout * taps * d.cin * 2 / 128;
        cuuint64_t dims[2] = {64, rows};
        cuuint64_t strides[1] = {128};
        cuuint32_t box[2] = {64, (cuuint32_t)(b_bytes / 128)};
        cuuint32_t estr[2] = {1, 1};
        if (enc(tmWp, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L.weight_halo, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
            tm_drop(&L.tm_b, 1, tmWp);
            return DC_ERR_CUDA;
        }
    }
    TcHaloArgs ha;
    TcArgs& a = ha.t;
    a.bias = L.bias; a.out = (__nv_bfloat16*)out; a.tile_list = tile_list; a.tile_count = tile_count; a.masks = masks;
    a.Ho = d.out_h; a.Wo = d.out_w; a.Co = d.cout; a.Ci = d.cin; a.kh = d.kh; a.kw = d.kw; a.sh = 1; a.sw = 1;
    a.ph = d.ph; a.pw = d.pw; a.relu = d.relu; a.tiles_x = L.tiles_x; a.tiles_y = L.tiles_y;
    a.BN = bn; a.NB = d.cout / bn; a.nb_off = 0; a.BK = 64; a.kchunks = kchunks; a.MT = 1; a.nbuf = 2;
    a.a_bytes = 0; a.b_bytes = b_bytes; a.sbo = 128; a.layout_type = 0;
    // instruction descriptor: D = f32, A = B = bf16, both K-major, N = bn, M = 256 (128 rows in each CTA)
    a.idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
    a.status = c->status;
    set_wait_limit(c, a);
    a.tmem_cols = tmem_cols_for(2, 1, bn);
    ha.wpacked = (const __nv_bfloat16*)L.weight_halo;
    ha.PW = DC_TILE_W; ha.PH = PH; ha.plane_bytes = 0;
    ha.patch_bytes = PH * DC_TILE_W * 128;                       // one slab
    const int budget = ring_budget(1);
    ha.a_stages = 2;
    for (int as = 4; as > 2; --as)
        if (budget - as * ha.patch_bytes >= 4 * b_bytes) { ha.a_stages = as; break; }
    int st = (budget - ha.a_stages * ha.patch_bytes) / b_bytes;
    a.stages = st > kMaxStages ? kMaxStages : st;
    if (a.stages < 2) return DC_ERR_CONFIG;
    a.bias_smem = t_bias_bytes ? d.cout : 0;
    const size_t smem = (size_t)ha.a_stages * ha.patch_bytes + (size_t)a.stages * b_bytes + ctl_bytes(4) + t_bias_bytes + 1280;
    if (smem > 227 * 1024) return DC_ERR_CONFIG;
    static dc_once_per_device attr_set;
    if (attr_set.first(c->device))
        DC_CUDA(cudaFuncSetAttribute(k_conv_tc_pair, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
    const long long items = (long long)(((max_tiles < 1 ? 1 : max_tiles) + 1) / 2) * a.NB;
    const int max_pairs = c->num_sms / 2;                        // one CTA per SM, a pair per TPC
    const int pairs = items > max_pairs ? max_pairs : (int)items;
    dc_prof_scope ps(c, DC_ST_CONV);
    DC_CUDA(launch_conv_kernel(k_conv_tc_pair, 2 * pairs, kThreads, smem, c->stream, *tmAp, *tmWp, ha));
    c->launches += 1;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}

static int launch_group(dc_cache* c, int layer, int grp, const void* in, void* out, const int32_t* tile_list,
                        const int32_t* tile_count, const uint32_t* masks, int max_tiles);

int dc_launch_conv_bf16(dc_cache* c, int layer, const void* in, void* out, const int32_t* tile_list,
                        const int32_t* tile_count, const uint32_t* masks, int max_tiles)
{
    const int G = n_groups(c->L[layer].d);
    t_ring_kb = c->overlap_mode ? 182 : 200;
    t_pdl = !c->overlap_mode;
    t_bias_bytes = bias_bytes_for(group_view(c->L[layer].d));
    // eight epilogue warps take the registers that the block search of the next frame needs to stay resident beside
    // this kernel: while that overlap is in use the CTA keeps to four
    t_epi_warps = c->L[layer].tc_ew == 8 && !c->overlap_mode ? 8 : 4;
    for (int grp = 0; grp < G; ++grp) {                           // a grouped layer: one launch per group
        int rc = launch_group(c, layer, grp, in, out, tile_list, tile_count, masks, max_tiles);
        if (rc == DC_ERR_CONFIG && t_ring_kb != 200) {            // the layer's tuned shape needs the full rings: it gets them
            t_ring_kb = 200;
            rc = launch_group(c, layer, grp, in, out, tile_list, tile_count, masks, max_tiles);
        }
        if (rc != DC_OK) return rc;
    }
    return DC_OK;
}

static int launch_group(dc_cache* c, int layer, int grp, const void* in, void* out, const int32_t* tile_list,
                        const int32_t* tile_count, const uint32_t* masks, int max_tiles)
{
    dc_layer_rt& L = c->L[layer];
    if (L.flat && L.tc_mt > 2) return DC_ERR_CONFIG;              // flat tiles exist in the tap-by-tap kernel only
    if (L.tc_mt == 7) return launch_pair(c, layer, in, out, tile_list, tile_count, masks, max_tiles);
    if (L.tc_mt >= 5) return launch_halo(c, layer, grp, L.tc_mt - 4, true, in, out, tile_list, tile_count, masks, max_tiles);
    if (L.tc_mt >= 3) return launch_halo(c, layer, grp, L.tc_mt - 2, false, in, out, tile_list, tile_count, masks, max_tiles);
    const bool grouped = n_groups(L.d) > 1;
    const bool pad16 = !grouped && pad16_ok(L.d) && L.weight_packed && L.in_padded;
    const dc_layer_desc d = pad16 ? padded16(L.d) : group_view(L.d);
    const int cin_all = pad16 ? 16 : L.d.cin, cout_all = L.d.cout;
    const void* weights = pad16 ? L.weight_packed : L.weight;
    if (pad16) {
        const size_t pixels = (size_t)c->S * L.in_h * L.in_w;
        int grid_pad = (int)((pixels + 255) / 256); if (grid_pad > c->num_sms * 8) grid_pad = c->num_sms * 8;
        dc_prof_scope ps(c, DC_ST_CONV);
        k_pad_channels16<<<grid_pad, 256, 0, c->stream>>>((const __nv_bfloat16*)in, pixels, L.d.cin, (__nv_bfloat16*)L.in_padded);
        c->launches += 1;
        in = L.in_padded;
    }
    in = (const uint8_t*)in + (size_t)grp * d.cin * 2;            // the group's first input channel (grp = 0 when ungrouped)
    TcPlan p;
    int ctas = L.tc_ctas == 2 ? 2 : 1;
    if (ctas == 2 && !make_plan(d, p, L.tc_mt, L.tc_bn, 2)) ctas = 1;
    if (!make_plan(d, p, L.tc_mt, L.tc_bn, ctas)) {
        if (smallc_ok(d)) return launch_smallc(c, layer, in, out, tile_list, tile_count, masks, max_tiles);
        return DC_ERR_CONFIG;
    }
    EncodeTiledFn enc = encode_fn();
    if (!enc) return DC_ERR_CUDA;
    bool hit_a, hit_b;
    CUtensorMap* tmAp = tm_find(L.tm_a, 4, &L.tm_next, in, L.flat ? 8 : 1, 0, &hit_a);
    CUtensorMap* tmBp = tm_find(&L.tm_b, 1, nullptr, weights, 1, p.BN, &hit_b);
    if (!hit_a) {   // input map [S][Hi][Wi][Ci] bf16; box = BK channels x 16 columns x 8 rows x 1 stream
        cuuint64_t dims[4] = {(cuuint64_t)d.cin, (cuuint64_t)L.in_w, (cuuint64_t)L.in_h, (cuuint64_t)c->S};
        cuuint64_t strides[3] = {(cuuint64_t)cin_all * 2, (cuuint64_t)L.in_w * cin_all * 2, (cuuint64_t)L.in_h * L.in_w * cin_all * 2};
        // a strided convolution reads every sw-th column / sh-th row: the box spans TW * sw x TH * sh input
        // pixels and the traversal strides pick TW x TH of them
        // (flat tiles: one image row of 8 pixels per box)
        cuuint32_t box[4] = {(cuuint32_t)p.BK, (cuuint32_t)(DC_TILE_W * d.sw), (cuuint32_t)(L.flat ? 1 : DC_TILE_H * d.sh), 1};
        cuuint32_t estr[4] = {1, (cuuint32_t)d.sw, (cuuint32_t)(L.flat ? 1 : d.sh), 1};
        if (enc(tmAp, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(in), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, p.swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) { tm_drop(L.tm_a, 4, tmAp); tm_drop(&L.tm_b, 1, tmBp); return DC_ERR_CUDA; }
    }
    if (!hit_b) {   // weights [cout][K] bf16, K = kh * kw * cin
        const cuuint64_t K = (cuuint64_t)d.kh * d.kw * d.cin;
        cuuint64_t dims[2] = {K, (cuuint64_t)cout_all};               // every group's rows; a launch reads its own (nb_off)
        cuuint64_t strides[1] = {K * 2};
        cuuint32_t box[2] = {(cuuint32_t)p.BK, (cuuint32_t)p.BN};
        cuuint32_t estr[2] = {1, 1};
        if (enc(tmBp, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(weights), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, p.swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) { tm_drop(&L.tm_b, 1, tmBp); return DC_ERR_CUDA; }
    }
    const CUtensorMap& tmA = *tmAp;
    const CUtensorMap& tmB = *tmBp;
    TcArgs a;
    a.bias = L.bias; a.out = (__nv_bfloat16*)out; a.tile_list = tile_list; a.tile_count = tile_count; a.masks = masks;
    a.Ho = d.out_h; a.Wo = d.out_w; a.Co = cout_all; a.Ci = d.cin; a.kh = d.kh; a.kw = d.kw; a.sh = d.sh; a.sw = d.sw;
    a.ph = d.ph; a.pw = d.pw; a.relu = d.relu; a.tiles_x = L.tiles_x; a.tiles_y = L.tiles_y;
    a.BN = p.BN; a.NB = p.NB; a.nb_off = grp * p.NB; a.BK = p.BK; a.kchunks = d.cin / p.BK; a.stages = p.stages; a.MT = p.MT; a.nbuf = p.nbuf;
    a.a_bytes = p.a_bytes; a.b_bytes = p.b_bytes; a.sbo = p.sbo; a.layout_type = p.layout_type;
    a.tmem_cols = tmem_cols_for(p.nbuf, p.MT, p.BN);
    // instruction descriptor: D = f32, A = B = bf16, both K-major, N = BN, M = 128
    a.idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.BN >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
    a.status = c->status;
    a.flat = L.flat; a.gpr = L.gpr; a.n_groups_all = c->S * d.out_h * L.gpr;
    a.epi_warps = epi_warps_for(ctas);
    a.bias_smem = t_bias_bytes ? d.cout : 0;
    set_wait_limit(c, a);
    static dc_once_per_device attr_set;
    if (attr_set.first(c->device)) {
        DC_CUDA(cudaFuncSetAttribute(k_conv_tc<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        DC_CUDA(cudaFuncSetAttribute(k_conv_tc<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
    }
    long long items = (long long)(((max_tiles < 1 ? 1 : max_tiles) + p.MT - 1) / p.MT) * p.NB;
    int grid = items > c->num_sms * ctas ? c->num_sms * ctas : (int)items;
    dc_prof_scope ps(c, DC_ST_CONV);
    if (p.MT == 2) DC_CUDA(launch_conv_kernel(k_conv_tc<2>, grid, threads_for(a.epi_warps), p.smem, c->stream, tmA, tmB, a));
    else DC_CUDA(launch_conv_kernel(k_conv_tc<1>, grid, threads_for(a.epi_warps), p.smem, c->stream, tmA, tmB, a));
    c->launches += 1;
    DC_CUDA(cudaGetLastError());
    return DC_OK;
}

// Picks, per convolution layer, the operand scheme and the work-item shape (tiles per item x channels per block)
// by timing the candidates once on the layer's own buffers with every tile dirty.  Within one scheme the choice
// changes only how the work is cut.  Between schemes the order in which the taps are accumulated in fp32 differs
// (the column-slab kernel goes column by column), so two choices can differ in the last bits of a bf16 output; every
// choice stays within the parity bound.  Called by dc_cache_create (which may synchronise).
int dc_conv_bf16_autotune(dc_cache* c, int layer, const void* in)
{
    dc_layer_rt& L = c->L[layer];
    TcPlan p;
    if (c->cfg.dtype != DC_BF16 || !encode_fn() || getenv("DC_NO_TENSOR_CORES")) return DC_OK;
    const bool grouped = n_groups(L.d) > 1;
    if (grouped && !dc_conv_bf16_supported(c, layer)) return DC_OK;
    const dc_layer_desc de = grouped ? group_view(L.d) : (pad16_ok(L.d) ? padded16(L.d) : L.d);
    const bool generic = make_plan(de, p);
    if (!generic && (grouped || !smallc_ok(L.d))) return DC_OK;
    if (getenv("DC_CONV_NO_TUNE")) return DC_OK;
    cudaEvent_t e0, e1;
    DC_CUDA(cudaEventCreate(&e0));
    DC_CUDA(cudaEventCreate(&e1));
    float best = 1e30f; int best_mt = L.tc_mt, best_bn = L.tc_bn, best_ctas = 1, best_flat = 0, best_ew = 4;
    constexpr int kTuneReps = 6;                                      // timed launches per candidate, after one untimed
    // the GPU may have been idle: bring the clocks up before the first candidate is timed
    for (int rep = 0; rep < 12; ++rep)
        if (dc_launch_conv_bf16(c, layer, in, L.map[0], L.all_list, dc_all_count(c, layer), c->zero_masks, dc_layer_tiles(c, L)) != DC_OK) break;
    const bool verbose = getenv("DC_VERBOSE") != nullptr;
    // times the launch the current L.tc_* fields select; keeps it when it is the fastest so far
    // DC_CONV_SCHEME=<code> (diagnostics, tests): only candidates of that operand scheme are timed, so the scheme runs
    // wherever it can (1, 2 tap by tap; 3, 4 patch; 5, 6 column slabs; the second of each pair with two tiles per item;
    // 7 column slabs on CTA pairs; 8, 9 tap by tap on flat tiles)
    const int only = getenv("DC_CONV_SCHEME") ? atoi(getenv("DC_CONV_SCHEME")) : 0;
    auto trial = [&](const char* what) {
        if (only > 0 && generic && (L.flat ? L.tc_mt + 7 : L.tc_mt) != only) return;
        int rc = DC_OK;
        for (int rep = 0; rep < kTuneReps + 1 && rc == DC_OK; ++rep) {
            if (rep == 1) cudaEventRecord(e0, c->stream);
            rc = dc_launch_conv_bf16(c, layer, in, L.map[0], L.all_list, dc_all_count(c, layer), c->zero_masks, dc_layer_tiles(c, L));
        }
        cudaEventRecord(e1, c->stream);
        if (rc != DC_OK || cudaEventSynchronize(e1) != cudaSuccess) { cudaGetLastError(); return; }
        float ms = 0.f;
        cudaEventElapsedTime(&ms, e0, e1);
        if (verbose) fprintf(stderr, "libdeepcache: layer %d: %s, tiles/item code %d, %d channels per block, %d CTA(s) per SM, %d epilogue warps: %.3f ms\n",
                             layer, what, L.flat ? L.tc_mt + 7 : L.tc_mt, L.tc_bn, L.tc_ctas, L.tc_ew, ms / kTuneReps);
        if (ms < best) { best = ms; best_mt = L.tc_mt; best_bn = L.tc_bn; best_ctas = L.tc_ctas; best_flat = L.flat; best_ew = L.tc_ew; }
    };
    // one CTA per SM with four or eight epilogue warps, or two CTAs per SM with four each
    for (int shape = 0; shape < 3; ++shape) {
        const int ctas = shape == 2 ? 2 : 1;
        L.tc_ctas = ctas; L.tc_ew = shape == 1 ? 8 : 4;
        t_epi_warps = L.tc_ew;                                        // make_plan below sizes the rings for it
        t_bias_bytes = bias_bytes_for(de);
        if (!generic) {                                               // few input channels: one kernel shape, 1 or 2 CTAs per SM
            if (ctas == 2 && tmem_cols_for(2, 1, L.d.cout) > 256) continue;
            trial("few-channel kernel");
            continue;
        }
        const int default_bn = p.BN;
        for (int bn = default_bn; bn >= 64 && bn >= default_bn / 2; bn -= 32) {
            if (de.cout % bn != 0) continue;
            for (int mt = 1; mt <= 2; ++mt) {
                TcPlan q;
                if (!make_plan(de, q, mt, bn, ctas)) continue;
                L.tc_mt = mt; L.tc_bn = bn;
                trial("tap-by-tap kernel");
                // flat tiles where the 16 x 8 blocks leave a good part of their pixels outside the map
                if (L.tiles_flat * 20 <= L.tiles_x * L.tiles_y * c->S * 19 || only >= 8) {
                    L.flat = 1;
                    trial("tap-by-tap kernel, flat tiles");
                    L.flat = 0;
                }
            }
        }
        HaloPlan h0;
        if (L.weight_halo && halo_ok(de, h0)) {
            for (int bn = h0.BN; bn >= 64 && bn >= h0.BN / 2; bn -= 32) {
                HaloPlan h;
                if (!halo_ok(de, h, bn)) continue;
                for (int mt = 1; mt <= 2; ++mt) {                      // tc_mt 3 / 4: patch-reuse kernel with 1 / 2 tiles per item
                    if (ctas == 2 && tmem_cols_for(mt * h.BN * 2 <= 512 ? 2 : 1, mt, h.BN) > 256) continue;
                    L.tc_bn = bn;
                    if (bn == h0.BN) { L.tc_mt = mt + 2; trial("patch-reuse kernel"); }
                    L.tc_mt = mt + 4;                                   // tc_mt 5 / 6: column slabs with 1 / 2 tiles per item
                    trial("column-slab kernel");
                }
            }
        }
    }
    {
        int pbn = 0;
        if (generic && L.weight_halo && pair_ok(L.d, pbn)) {          // tc_mt 7: a CTA pair per two tiles (cta_group::2)
            L.tc_mt = 7; L.tc_bn = pbn; L.tc_ctas = 1; L.tc_ew = 4;
            trial("CTA-pair kernel");
        }
    }
    L.tc_mt = best_mt; L.tc_bn = best_bn; L.tc_ctas = best_ctas; L.flat = best_flat; L.tc_ew = best_ew;
    cudaEventDestroy(e0); cudaEventDestroy(e1);
    c->launches = 0;
    if (verbose) fprintf(stderr, "libdeepcache: layer %d: chose code %d, %d channels per block, %d CTA(s) per SM, %d epilogue warps (%.3f ms)\n",
                         layer, best_flat ? best_mt + 7 : best_mt, best_bn, best_ctas, best_ew, best / kTuneReps);
    return DC_OK;
}

// Failure detection without a fault (not part of the public header: tests declare it themselves).  The next
// tensor-core convolution launch of this cache issues none of its operand copies and bounds its waits by wait_ms
// instead of 2 s: the MMA and epilogue roles find nothing arriving, give up, record DC_ERR_TIMEOUT in the status
// word, free their tensor memory and the kernel returns normally.  No copy and no MMA is in flight when they leave.
// The launch after it is an ordinary one.
extern "C" int dc_debug_stall_next_conv(dc_cache* c, int wait_ms)
{
    if (!c || wait_ms < 1 || wait_ms > 1000) return DC_ERR_ARG;
    c->debug_stall_ms = wait_ms;
    return DC_OK;
}
