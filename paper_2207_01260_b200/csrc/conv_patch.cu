// Stride-1 dense conv task (3x3 and other R x S > 1) on the sm_100a tensor cores with the input
// patch kept in shared memory (paper Sec. 3.4: a task is Conv2d + folded BatchNorm + activation;
// Sec. 3.5: the filter count is whatever pruning left).
//
// Why a second tensor-core kernel: the im2col kernel (conv_tc.cu) writes every activation element
// R*S times into shared memory, and on this GPU the shared-memory port (128 bytes per clock: TMA
// writes plus the operand reads of tcgen05.mma) is what bounds it, not the tensor pipe.  Here a
// tile is TH whole output rows of one image.  Its input patch, (TH + R - 1) x (W + 2 pad) pixels x
// 64 channels, is loaded ONCE per channel block by one tiled TMA load (out-of-range pixels and
// channels arrive as zeros, which is the padding).  The patch sits in shared memory as rows of
// 128 bytes, one per pixel, in row-major order of the padded image, 128-byte swizzled.  For filter
// tap (r, s) the pixel operand of the MMA is the same patch read from a start address
// (r * Wp + s) * 128 bytes further on (Wp = W + 2 pad): the swizzle is a function of the
// shared-memory address, so a descriptor may start at any 128-byte row (checked on B200).
//
// The accumulator row of a pixel is its "slot" i * Wp + j (i row in the tile, j column); slots with
// j >= Q are the S - 1 wrap-around columns: they are computed and thrown away.  A tile has MT
// blocks of 128 slots (MT = 1 or 2, one accumulator each, both fed by the same filter stage).
//
//   warp 0       patch loads (one per channel block); with a residual, one more load per group of
//                64 filters brings the residual tile in through the same ring;
//   warps 1, 2   filter loads, one per (channel block, tap), taken in turn; small filter sets
//                stay resident in shared memory for the whole kernel;
//   warps 3, 12  tcgen05.mma issue, one warp per accumulator block; the residual tile is added by
//                one more MMA against a 64 x 64 identity held in shared memory (bf16 x 1.0 into an
//                fp32 accumulator is exact), so the epilogue never touches global memory for it
//                (the 1x1 instantiation, whose tile is flat, still adds it in the epilogue);
//   warps 4..11  epilogue: tcgen05.ld, bias, activation, bf16 into a swizzled staging
//                buffer, then ONE TMA store per group of 64 filters whose box is the tile's rows x
//                Wp pixels (wrap-around columns, rows below the image and filters beyond k_pad lie
//                outside the tensor map and are not written).  With a fused max-pool the staged
//                tile is pooled and copied out by hand instead, eight threads per output pixel.
// Every wait is bounded (see sm100_ptx.cuh); on expiry the CTA raises STATUS_TIMEOUT and leaves.
#include <cuda.h>

#include <cstdlib>
#include <cstring>
#include <mutex>

#include "common.cuh"
#include "plan.h"
#include "sm100_ptx.cuh"

namespace cprune {

constexpr int PK_THREADS = 13 * 32;       // general kernel: 5 role warps + 8 epilogue warps
constexpr int PK_THREADS_DENSE = 21 * 32; // dense-staging kernel: 16 epilogue warps (its epilogue bounds the tile; it needs few registers)
constexpr int PK_POOL_WARPS = 8;          // 3x3-pool kernel: these warps pool the staged tile while the epilogue warps stage the next one
constexpr int PK_THREADS_POOL3 = (13 + PK_POOL_WARPS) * 32;
// kernel instantiations
constexpr int PK_GENERAL = 0, PK_DENSE = 1, PK_POOL3 = 2;
__host__ __device__ constexpr int pk_threads(int mode) { return mode == PK_DENSE ? PK_THREADS_DENSE : (mode == PK_POOL3 ? PK_THREADS_POOL3 : PK_THREADS); }
__host__ __device__ constexpr int pk_epi_warps(bool dense) { return dense ? 16 : 8; }
constexpr int PK_MMA_WARP = 3;
constexpr int PK_FIRST_EPI = 4;
// (the warp after the epilogue warps issues for the second accumulator block when MT = 2)
constexpr int PK_MAX_WSTAGES = 32;
constexpr int PK_MAX_PATCH_STAGES = 4;   // patch ring: 2 stages, more for tasks with small patches and several channel blocks
constexpr int PK_CTRL_BYTES = 5120;      // barriers (1 KB) + slot table (2 KB) + bias (2 KB)
constexpr int PK_BIAS_FLOATS = 512;      // the task's bias is kept in shared memory when it has at most this many filters
constexpr int PK_BLOCK_BYTES = 16384;    // staged block: 128 slots x 64 filters bf16
constexpr int PK_IDENT_BYTES = 8192;     // 64 x 64 identity (bf16, 128-byte rows): filter-side operand that adds a residual block

struct PatchParams {
    int P, Q, Wp, TH, tiles_per_img, tiles_m, tiles_n;
    int TW, tiles_w, step_h, step_w, org;   // tile (ty, tx) starts at output (ty * step_h + org, tx * step_w + org) and spans TH x TW
    int out_h, out_w;                       // stored extent (after a fused pool)
    int FT, MT, R, S, pad, pad_w, cblks, ksteps_last, k_pad;   // pad: rows above the image in a patch; pad_w: columns left of it
    int act, wstages, pstages, resident, acc_bufs, staging_bufs, pool;
    int patch_bytes;       // shared memory of one patch stage
    int patch_box_bytes;   // bytes one patch load delivers
    int w_stage_bytes;     // shared memory of one filter stage (FT rows, rounded up to 1024 bytes)
    int rb16;              // bytes per pixel row in shared memory / 16: 8 (64 channels) or 2 (16 channels, regrouped stems)
    int dense;             // the staged tile is [slot][k_pad] as in memory and leaves by one bulk copy (flat tasks, one filter tile)
    int dense_pitch;       // ... bytes per slot in the staging buffer: k_pad * 2, or 16 more (then the tile leaves by a tiled copy)
    int stage_bytes;       // shared memory of one staging buffer
    int res_blocks;        // residual added on the tensor core: 64-filter blocks of the residual tile per item (0: none)
    const float *bias;
    const __nv_bfloat16 *res;
    __nv_bfloat16 *y;
    int *status;
};

// Maximum of 8 non-negative bf16 values (after ReLU / ReLU6; max.f32 never yields -0): their bit patterns order like
// unsigned integers, so one SIMD integer instruction handles two values.
__device__ __forceinline__ uint4 bf16x8_max_nonneg(uint4 a, uint4 b) {
    return make_uint4(__vmaxu2(a.x, b.x), __vmaxu2(a.y, b.y), __vmaxu2(a.z, b.z), __vmaxu2(a.w, b.w));
}

__device__ __forceinline__ uint4 bf16x8_max(uint4 a, uint4 b) {
    uint4 r;
    __nv_bfloat162 *pa = reinterpret_cast<__nv_bfloat162 *>(&a), *pb = reinterpret_cast<__nv_bfloat162 *>(&b);
    __nv_bfloat162 *pr = reinterpret_cast<__nv_bfloat162 *>(&r);
#pragma unroll
    for (int i = 0; i < 4; ++i) pr[i] = __hmax2(pa[i], pb[i]);
    return r;
}

// All MMAs of one filter tap for one accumulator block: nk steps of 16 channels.  a_lo and w_lo are
// the low words of the operand descriptors (start address in 16-byte units).  Called by the whole warp: the
// operands are computed by all lanes (they stay in uniform registers) and one elected lane issues.
__device__ __forceinline__ void issue_tap(uint32_t d_tmem, uint32_t a_lo, uint32_t w_lo, uint32_t desc_hi, uint32_t idesc,
                                          uint32_t accumulate, int nk, uint32_t commit_w, uint32_t commit_p) {
    uint32_t al[4], wl[4];
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) { wl[kk] = w_lo + (uint32_t)(2 * kk); al[kk] = a_lo + (uint32_t)(2 * kk); }
    if (elect_one()) {
        if (nk == 4) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) umma_bf16_words(d_tmem, al[kk], wl[kk], desc_hi, idesc, kk ? 1u : accumulate);
        } else {
            umma_bf16_words(d_tmem, al[0], wl[0], desc_hi, idesc, accumulate);
#pragma unroll
            for (int kk = 1; kk < 3; ++kk)
                if (kk < nk) umma_bf16_words(d_tmem, al[kk], wl[kk], desc_hi, idesc, 1u);
        }
        if (commit_w) umma_commit(commit_w);
        if (commit_p) umma_commit(commit_p);
    }
    __syncwarp();
}

// A whole filter row (S taps) from one elected block: used when nothing has to be waited for between taps.
__device__ __forceinline__ void issue_row(uint32_t d_tmem, uint32_t a_lo, uint32_t w_lo, uint32_t desc_hi, uint32_t idesc,
                                          uint32_t accumulate, int nk, int S, uint32_t slot_step, uint32_t w_step, uint32_t commit_p) {
    if (elect_one()) {
        for (int s = 0; s < S; ++s) {
            if (nk == 4) {
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    umma_bf16_words(d_tmem, a_lo + (uint32_t)(2 * kk), w_lo + (uint32_t)(2 * kk), desc_hi, idesc, kk ? 1u : accumulate);
            } else {
                umma_bf16_words(d_tmem, a_lo, w_lo, desc_hi, idesc, accumulate);
#pragma unroll
                for (int kk = 1; kk < 3; ++kk)
                    if (kk < nk) umma_bf16_words(d_tmem, a_lo + (uint32_t)(2 * kk), w_lo + (uint32_t)(2 * kk), desc_hi, idesc, 1u);
            }
            accumulate = 1;
            a_lo += slot_step;
            w_lo += w_step;
        }
        if (commit_p) umma_commit(commit_p);
    }
    __syncwarp();
}

// First output pixel (may be -1 with the 3x3 pool, whose windows reach one pixel outside the tile's own pooled
// pixels) and image of tile tm.
__device__ __forceinline__ void tile_origin(const PatchParams &p, int tm, int &n, int &p0, int &q0) {
    n = tm / p.tiles_per_img;
    const int r = tm - n * p.tiles_per_img;
    int ty = r, tx = 0;
    if (p.tiles_w > 1) { ty = r / p.tiles_w; tx = r - ty * p.tiles_w; }
    p0 = ty * p.step_h + p.org;
    q0 = tx * p.step_w + p.org;
}

template <int MODE>
__global__ void __launch_bounds__(pk_threads(MODE), 1)
conv_patch_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
                  const __grid_constant__ CUtensorMap tm_y, const __grid_constant__ CUtensorMap tm_res, const PatchParams p) {
    extern __shared__ uint8_t smem_raw[];
    constexpr bool DENSE = MODE == PK_DENSE;
    constexpr bool SPLIT = MODE == PK_POOL3;      // staging by the epilogue warps, pooling by PK_POOL_WARPS further warps
    constexpr int EPI_WARPS = pk_epi_warps(DENSE);
    constexpr int MMA_WARP2 = PK_FIRST_EPI + EPI_WARPS;
    pdl_trigger();
    if (threadIdx.x == 0) {
        // the descriptors are fetched on first use otherwise, which the first loads would wait for
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_x) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_w) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_y) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_res) : "memory");
    }
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - raw);
    const uint32_t w_bytes = (uint32_t)p.w_stage_bytes;                   // stage stride
    const uint32_t w_tx_bytes = (uint32_t)p.FT * 16u * (uint32_t)p.rb16;  // bytes one filter load delivers
    const uint32_t patch0 = base;
    const uint32_t w0 = patch0 + (uint32_t)p.pstages * (uint32_t)p.patch_bytes;
    const uint32_t staging0 = w0 + (uint32_t)p.wstages * w_bytes;
    const uint32_t stage_buf_bytes = (uint32_t)p.stage_bytes;
    const uint32_t ident0 = staging0 + (uint32_t)p.staging_bufs * stage_buf_bytes;   // present when res_blocks > 0
    const uint32_t ctrl0 = ident0 + (p.res_blocks ? (uint32_t)PK_IDENT_BYTES : 0u);
    uint8_t *ctrl = smem + (ctrl0 - base);
    auto pfull = [&](int s) { return ctrl0 + 8u * s; };
    auto pempty = [&](int s) { return ctrl0 + 32u + 8u * s; };
    auto tfull = [&](int a) { return ctrl0 + 64u + 8u * a; };
    auto tempty = [&](int a) { return ctrl0 + 80u + 8u * a; };
    const uint32_t epi_bar = ctrl0 + 96u;
    auto res_full = [&](int b) { return ctrl0 + 112u + 8u * b; };   // residual tile landed in staging buffer b
    uint32_t *tmem_slot = (uint32_t *)(ctrl + 104);
    volatile int *abort_flag = (volatile int *)(ctrl + 108);
    auto sfull = [&](int b) { return ctrl0 + 640u + 8u * b; };      // 3x3-pool kernel: staging buffer b holds a finished group
    auto sempty = [&](int b) { return ctrl0 + 656u + 8u * b; };     // ... has been pooled and may be overwritten
    auto wfull = [&](int s) { return ctrl0 + 128u + 8u * s; };
    auto wempty = [&](int s) { return ctrl0 + 384u + 8u * s; };
    int2 *lut = (int2 *)(ctrl + 1024);   // entry -> (source slot | tile row << 16, output offset in elements); x < 0: nothing to store

    // the shuffle tells the compiler that the warp number is the same in all lanes, so that the role code below
    // (loop counters, descriptors, TMA coordinates) can live in uniform registers
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    const int RS = p.R * p.S;

    // barrier set-up, spread over the lanes of warp 0 (one thread doing up to 70 initialisations costs microseconds).
    // Every accumulator block has its own issuing warp: stages are free, and a tile is complete, once all have committed.
    if (threadIdx.x < 32) {
        const int l = threadIdx.x;
        if (l < p.pstages) { mbar_init(pfull(l), 1); mbar_init(pempty(l), p.MT); }
        if (l < 2) { mbar_init(tfull(l), p.MT); mbar_init(tempty(l), EPI_WARPS); mbar_init(res_full(l), 1); }
        if (l == 2) { mbar_init(epi_bar, EPI_WARPS); *abort_flag = 0; }
        if (SPLIT && l >= 4 && l < 6) { mbar_init(sfull(l - 4), EPI_WARPS); mbar_init(sempty(l - 4), PK_POOL_WARPS); }
        if (l < p.wstages) { mbar_init(wfull(l), 1); mbar_init(wempty(l), p.MT); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // the bias (written when the task was packed, not by the preceding kernel) in shared memory: a read costs the
    // epilogue a fraction of what the same read through L1 does
    // (the epilogue warps copy it while the first tile is being computed: see there)
    float *bias_s = (float *)(ctrl + 3072);
    const int k_all = p.tiles_n * p.FT;
    const bool bias_staged = k_all <= PK_BIAS_FLOATS;
    const float *bias_src = bias_staged ? bias_s : p.bias;
    // 64 x 64 identity in the layout of a filter stage (128-byte rows, 128-byte swizzle): row r holds 1.0 at channel r
    if (p.res_blocks) {
        uint8_t *ident = smem + (ident0 - base);
        for (int e = threadIdx.x; e < 64 * 8; e += blockDim.x) {
            const int r = e >> 3, c = e & 7;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (c == (r >> 3)) {
                const uint32_t one = (r & 1) ? 0x3F800000u : 0x00003F80u;      // bf16 1.0 in the odd or even half
                const int word = (r & 7) >> 1;
                if (word == 0) v.x = one; else if (word == 1) v.y = one; else if (word == 2) v.z = one; else v.w = one;
            }
            *(uint4 *)(ident + sub_off(r, c)) = v;
        }
        fence_async_smem();
    }
    // slot table: which accumulator rows hold real output pixels and where they go
    for (int e = threadIdx.x; e < 256 && p.pool == 1; e += blockDim.x) {
        int2 v = make_int2(-1, 0);
        {
            const int hq = p.Q >> 1;
            const int i2 = e / hq, j2 = e - i2 * hq;
            if (i2 < (p.TH >> 1)) v = make_int2((2 * i2 * p.Wp + 2 * j2) | ((2 * i2) << 16), (i2 * hq + j2) * p.k_pad);
        }
        lut[e] = v;
    }
    if (warp == PK_MMA_WARP) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // Set-up done.  Only the patch (and residual) loads of warp 0 read what the preceding kernel wrote, and everything
    // else in this kernel follows from them, so warp 0 alone waits for the predecessor; filters and bias were written
    // when the task was packed and are fetched right away.
    const uint32_t tmem_base = *tmem_slot;
    const int total_items = p.tiles_m * p.tiles_n;

    if (warp == 0) {
        // ------------------------------------------------------------------ patch loads
        pdl_wait();
        int ps = 0;
        uint32_t pphase = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
            int tm = item, nt = 0;
            if (p.tiles_n > 1) { tm = item / p.tiles_n; nt = item - tm * p.tiles_n; }
            int n, p0, q0;
            tile_origin(p, tm, n, p0, q0);
            for (int cb = 0; cb < p.cblks; ++cb) {
                ok = __all_sync(0xffffffffu, mbar_wait(pempty(ps), pphase ^ 1u, abort_flag, p.status));
                if (!ok) break;
                if (elect_one()) {
                    mbar_expect_tx(pfull(ps), (uint32_t)p.patch_box_bytes);
                    tma_load_4d(patch0 + (uint32_t)ps * p.patch_bytes, &tm_x, pfull(ps), cb * 64, q0 - p.pad_w, p0 - p.pad, n);
                }
                __syncwarp();
                if (++ps == p.pstages) { ps = 0; pphase ^= 1u; }
            }
            // The residual tile goes through the same ring, 64 filters at a time: its box is the tile's TH x Wp output
            // pixels, so pixel (i, j) lands in the row of slot i * Wp + j (wrap-around columns read as zero), and the MMA
            // warps add it to the accumulator by multiplying it with the identity.
            for (int j = 0; j < p.res_blocks && ok; ++j) {
                ok = __all_sync(0xffffffffu, mbar_wait(pempty(ps), pphase ^ 1u, abort_flag, p.status));
                if (!ok) break;
                if (elect_one()) {
                    mbar_expect_tx(pfull(ps), (uint32_t)(p.TH * p.Wp * 128));
                    tma_load_4d(patch0 + (uint32_t)ps * p.patch_bytes, &tm_res, pfull(ps), nt * p.FT + j * 64, q0, p0, n);
                }
                __syncwarp();
                if (++ps == p.pstages) { ps = 0; pphase ^= 1u; }
            }
        }
    } else if (warp < PK_MMA_WARP) {
        // ------------------------------------------------------------------ filter loads
        int ws = 0, turn = 0;
        uint32_t wphase = 0;
        bool ok = true;
        const int me = warp - 1;
        for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
            if (p.resident && item != (int)blockIdx.x) break;     // the filters of the first tile stay
            int nt = 0;
            if (p.tiles_n > 1) nt = item % p.tiles_n;
            const int k0 = nt * p.FT;
            for (int cb = 0; cb < p.cblks && ok; ++cb) {
                for (int tap = 0; tap < RS; ++tap) {
                    const bool mine = turn == me;
                    turn ^= 1;
                    if (mine) {
                        if (!p.resident) ok = __all_sync(0xffffffffu, mbar_wait(wempty(ws), wphase ^ 1u, abort_flag, p.status));
                        if (!ok) break;
                        if (elect_one()) {
                            mbar_expect_tx(wfull(ws), w_tx_bytes);
                            tma_load_3d(w0 + (uint32_t)ws * w_bytes, &tm_w, wfull(ws), cb * 64, tap, k0);
                        }
                        __syncwarp();
                    }
                    if (++ws == p.wstages) { ws = 0; wphase ^= 1u; }
                }
            }
        }
    } else if (warp == PK_MMA_WARP || warp == MMA_WARP2) {
        // ------------------------------------------------------------------ MMA issue
        // tcgen05.mma issue is close to synchronous (about two instructions may be pending, measured), so the
        // bookkeeping between taps would leave the tensor pipe idle if one warp issued everything: with MT = 2
        // each accumulator block gets its own issuing warp and the two interleave.
        const int mb = warp == PK_MMA_WARP ? 0 : 1;
        if (mb < p.MT) {
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.FT >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        int ps = 0, ws = 0, acc = 0;
        uint32_t pphase = 0, wphase = 0, acc_phase = 0;
        bool ok = true;
        // A lone warp pays several cycles for every instruction, so the loop works on the low descriptor words
        // only (32-bit adds) and issues a tap's MMAs from fully unrolled code.
        const uint32_t patch_lo0 = desc_lo(patch0), w_lo0 = desc_lo(w0);
        const uint32_t desc_hi = p.rb16 == 8 ? DESC_HI_SW128 : DESC_HI_SW32;
        const uint32_t slot_step = (uint32_t)p.rb16;                    // descriptor units (16 bytes) per pixel row
        const uint32_t patch_step = (uint32_t)p.patch_bytes >> 4, w_step = w_bytes >> 4;
        const uint32_t row_step = (uint32_t)(p.Wp - p.S + 1) * slot_step;   // from tap (r, S-1) to (r+1, 0)
        uint32_t patch_lo = patch_lo0, w_lo = w_lo0;
        for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
            ok = __all_sync(0xffffffffu, mbar_wait(tempty(acc), acc_phase ^ 1u, abort_flag, p.status));
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)((acc * p.MT + mb) * p.FT);
            uint32_t accumulate = 0;
            for (int cb = 0; cb < p.cblks && ok; ++cb) {
                ok = __all_sync(0xffffffffu, mbar_wait(pfull(ps), pphase, abort_flag, p.status));
                if (!ok) break;
                const int nk = cb == p.cblks - 1 ? p.ksteps_last : 4;
                uint32_t tap_lo = patch_lo + (uint32_t)(mb * 128) * slot_step;      // the second block's slots follow the first's
                if (p.resident && item != (int)blockIdx.x) {
                    // resident filters, loaded during the first tile: nothing to wait for, a filter row per elected block
                    for (int r = 0; r < p.R; ++r) {
                        issue_row(d_tmem, tap_lo, w_lo, desc_hi, idesc, accumulate, nk, p.S, slot_step, w_step, r == p.R - 1 ? pempty(ps) : 0u);
                        accumulate = 1;
                        tap_lo += (uint32_t)p.Wp * slot_step;
                        w_lo += (uint32_t)p.S * w_step;
                        ws += p.S;
                        if (ws == p.wstages) { ws = 0; w_lo = w_lo0; }
                    }
                } else {
                    int s = 0;
                    for (int tap = 0; tap < RS; ++tap) {
                        ok = __all_sync(0xffffffffu, mbar_wait(wfull(ws), p.resident ? 0u : wphase, abort_flag, p.status));
                        if (!ok) break;
                        {
                            const uint32_t cw = p.resident ? 0u : wempty(ws), cp = tap == RS - 1 ? pempty(ps) : 0u;
                            issue_tap(d_tmem, tap_lo, w_lo, desc_hi, idesc, accumulate, nk, cw, cp);
                        }
                        accumulate = 1;
                        w_lo += w_step;
                        if (++ws == p.wstages) { ws = 0; wphase ^= 1u; w_lo = w_lo0; }
                        tap_lo += slot_step;
                        if (++s == p.S) { s = 0; tap_lo += row_step - slot_step; }
                    }
                }
                patch_lo += patch_step;
                if (++ps == p.pstages) { ps = 0; pphase ^= 1u; patch_lo = patch_lo0; }
            }
            // residual blocks: accumulator columns 64 j .. += residual tile (slots x 64 filters) x identity (bf16 values
            // times 1.0, accumulated in float32: exact)
            for (int j = 0; j < p.res_blocks && ok; ++j) {
                ok = __all_sync(0xffffffffu, mbar_wait(pfull(ps), pphase, abort_flag, p.status));
                if (!ok) break;
                const int nres = min(64, p.FT - j * 64);
                const uint32_t idesc_r = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(nres >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
                issue_tap(d_tmem + (uint32_t)(j * 64), patch_lo + (uint32_t)(mb * 128) * slot_step, desc_lo(ident0), DESC_HI_SW128, idesc_r, 1u,
                          nres >> 4, 0u, pempty(ps));
                patch_lo += patch_step;
                if (++ps == p.pstages) { ps = 0; pphase ^= 1u; patch_lo = patch_lo0; }
            }
            if (ok && elect_one()) umma_commit(tfull(acc));
            __syncwarp();
            if (p.acc_bufs == 2) { if (++acc == 2) { acc = 0; acc_phase ^= 1u; } }
            else acc_phase ^= 1u;
        }
        }
    } else if (SPLIT && warp > MMA_WARP2) {
        // ------------------------------------------------------------------ 3x3 stride-2 pooling of staged groups
        // The tile computed conv rows p0 .. p0 + TH - 1 (p0 odd or -1) and holds the windows of (TH - 1) / 2 x (TW - 1) / 2
        // pooled pixels, all nine slots of each inside the staged tile.  A thread handles up to 512 / (32 * PK_POOL_WARPS) (pooled pixel,
        // 8 filters) items, the same ones in every tile: the shared-memory offsets of their window slots are worked out once.
        const int ctid = threadIdx.x - (MMA_WARP2 + 1) * 32;
        constexpr int ITEMS = 512 / (PK_POOL_WARPS * 32);
        const int groups = (p.FT + 63) / 64;
        const int tpc = (p.TW - 1) >> 1;
        const int n_entries = ((p.TH - 1) >> 1) * tpc;
        const bool clamp_lo = p.act != CPRUNE_ACT_NONE;
        uint32_t win_off[ITEMS][9];
        int win_pi[ITEMS], win_pj[ITEMS];
#pragma unroll
        for (int it = 0; it < ITEMS; ++it) {
            const int e = ctid + it * (PK_POOL_WARPS * 32);
            const int ent = e >> 3, chunk = e & 7;
            win_pi[it] = ent / tpc; win_pj[it] = ent - win_pi[it] * tpc;
#pragma unroll
            for (int k = 0; k < 9; ++k) {
                const int sl = (2 * win_pi[it] + k / 3) * p.Wp + 2 * win_pj[it] + k % 3;
                win_off[it][k] = (uint32_t)((sl >> 7) * PK_BLOCK_BYTES) + sub_off(sl & 127, chunk);
            }
        }
        uint32_t counter = 0;
        bool ok = true;
        // pixels outside the image never win: after ReLU / ReLU6 every value is >= 0 (and every window holds a real
        // pixel), so they can be replaced by 0 and the maximum taken on the bit patterns; else by -inf
        const uint4 fill = clamp_lo ? make_uint4(0u, 0u, 0u, 0u) : make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
        for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
            int tm = item, nt = 0;
            if (p.tiles_n > 1) { tm = item / p.tiles_n; nt = item - tm * p.tiles_n; }
            int n, p0, q0;
            tile_origin(p, tm, n, p0, q0);
            const int pr0 = (p0 + 1) >> 1, pc0 = (q0 + 1) >> 1;
            for (int g = 0; g < groups && ok; ++g) {
                const uint32_t b = counter & 1u;
                ok = __all_sync(0xffffffffu, mbar_wait(sfull(b), (counter >> 1) & 1u, abort_flag, p.status));
                if (!ok) break;
                const uint8_t *buf = smem + (staging0 - base) + b * stage_buf_bytes;
                const int kg = nt * p.FT + g * 64;
#pragma unroll
                for (int it = 0; it < ITEMS; ++it) {
                    const int e = ctid + it * (PK_POOL_WARPS * 32);
                    const int chunk = e & 7;
                    const int pr = pr0 + win_pi[it], pc = pc0 + win_pj[it];
                    if (e < n_entries * 8 && pr < p.out_h && pc < p.out_w && g * 64 + chunk * 8 < p.FT && kg + chunk * 8 < p.k_pad) {
                        const int r0 = p0 + 2 * win_pi[it], c0 = q0 + 2 * win_pj[it];
                        // bit d of a mask: window row / column d lies inside the image
                        const uint32_t rmask = (r0 >= 0 ? 1u : 0u) | 2u | (r0 + 2 < p.P ? 4u : 0u);
                        const uint32_t cmask = (c0 >= 0 ? 1u : 0u) | 2u | (c0 + 2 < p.Q ? 4u : 0u);
                        uint4 w[9];
#pragma unroll
                        for (int k = 0; k < 9; ++k) {
                            const uint4 t = *(const uint4 *)(buf + win_off[it][k]);
                            w[k] = ((rmask >> (k / 3)) & (cmask >> (k % 3)) & 1u) ? t : fill;
                        }
                        uint4 m;
                        if (clamp_lo) {
                            const uint4 a0 = bf16x8_max_nonneg(bf16x8_max_nonneg(w[0], w[1]), bf16x8_max_nonneg(w[2], w[3]));
                            const uint4 a1 = bf16x8_max_nonneg(bf16x8_max_nonneg(w[4], w[5]), bf16x8_max_nonneg(w[6], w[7]));
                            m = bf16x8_max_nonneg(bf16x8_max_nonneg(a0, a1), w[8]);
                        } else {
                            const uint4 a0 = bf16x8_max(bf16x8_max(w[0], w[1]), bf16x8_max(w[2], w[3]));
                            const uint4 a1 = bf16x8_max(bf16x8_max(w[4], w[5]), bf16x8_max(w[6], w[7]));
                            m = bf16x8_max(bf16x8_max(a0, a1), w[8]);
                        }
                        *(uint4 *)(p.y + (((size_t)n * p.out_h + pr) * p.out_w + pc) * p.k_pad + kg + chunk * 8) = m;
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(sempty(b));
                ++counter;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        const int quarter = warp & 3;
        const int half = (warp - PK_FIRST_EPI) >> 2;
        const int trow = quarter * 32 + lane;          // accumulator lane = slot within its 128-slot block
        const int etid = threadIdx.x - PK_FIRST_EPI * 32;
        int acc = 0;
        uint32_t acc_phase = 0, epi_phase = 0, group_counter = 0;
        bool ok = true;
        auto epi_sync = [&]() {
            __syncwarp();
            if (lane == 0) mbar_arrive(epi_bar);
            bool r = __all_sync(0xffffffffu, mbar_wait(epi_bar, epi_phase, abort_flag, p.status, false));
            epi_phase ^= 1u;
            return r;
        };
        // the task's bias into shared memory, while the first tile is being computed
        if (bias_staged) {
            for (int e = etid; e < k_all; e += EPI_WARPS * 32) bias_s[e] = __ldg(p.bias + e);
            ok = epi_sync();
        }
        // activation as a clamp: no branches in the per-element code
        const float act_lo = p.act == CPRUNE_ACT_NONE ? -INFINITY : 0.f, act_hi = p.act == CPRUNE_ACT_RELU6 ? 6.f : INFINITY;
        const bool clamp_lo = p.act != CPRUNE_ACT_NONE;      // results are >= 0
        const bool store_thread = warp == PK_FIRST_EPI && lane == 0;
        const int groups = (p.FT + 63) / 64;
        // one group and one filter tile: a thread stages the same 32 filters in every tile and keeps their bias in registers
        const bool bias_const = !DENSE && groups == 1 && p.tiles_n == 1;
        float bias_r[32];
        if (bias_const) {
#pragma unroll
            for (int j = 0; j < 32; ++j) bias_r[j] = (half * 32 + j < p.FT) ? __ldg(p.bias + half * 32 + j) : 0.f;
        }
        const int n_entries = p.pool == 1 ? (p.TH >> 1) * (p.Q >> 1) : ((p.TH - 1) >> 1) * ((p.TW - 1) >> 1);
        // 3x3 pool: a thread copies out at most two (pooled pixel, 8 filters) items per tile, the same ones in every tile;
        // the shared-memory offsets of their nine window slots are worked out once
        uint32_t win_off[2][9];
        int win_pi[2] = {0, 0}, win_pj[2] = {0, 0};
        if (MODE == PK_GENERAL && p.pool == 2) {
            const int tpc = (p.TW - 1) >> 1;
#pragma unroll
            for (int it = 0; it < 2; ++it) {
                const int e = etid + it * 256;
                const int ent = e >> 3, chunk = e & 7;
                win_pi[it] = ent / tpc; win_pj[it] = ent - win_pi[it] * tpc;
#pragma unroll
                for (int k = 0; k < 9; ++k) {
                    const int sl = (2 * win_pi[it] + k / 3) * p.Wp + 2 * win_pj[it] + k % 3;
                    win_off[it][k] = (uint32_t)((sl >> 7) * PK_BLOCK_BYTES) + sub_off(sl & 127, chunk);
                }
            }
        }
        // Residuals.  Everywhere but with dense staging the MMA warps add the residual on the tensor core (see there) and
        // the epilogue has nothing to do with it.  Dense staging: the residual of tile item_ (tiles_n == 1, one row of
        // tiles) is one contiguous range of memory, arrives in the staging buffer the tile will use and is added in place.
        const bool with_res = DENSE && p.res != nullptr;
        const bool dense_tiled = DENSE && p.dense_pitch != p.k_pad * 2;
        auto load_residual_dense = [&](int item_, uint32_t counter) {
            const int q0_ = item_ * p.step_w;
            const uint32_t bytes = (uint32_t)min(p.TW, p.Q - q0_) * (uint32_t)p.k_pad * 2u;
            const uint32_t b = counter & 1u;
            if (dense_tiled) {
                // the box is the whole tile, one piece wider than the tensor: what lies outside arrives as zeros
                mbar_expect_tx(res_full(b), (uint32_t)p.TW * (uint32_t)p.dense_pitch);
                tma_load_4d(staging0 + b * stage_buf_bytes, &tm_res, res_full(b), 0, q0_, 0, 0);
            } else {
                mbar_expect_tx(res_full(b), bytes);
                bulk_load(staging0 + b * stage_buf_bytes, p.res + (size_t)q0_ * p.k_pad, bytes, res_full(b));
            }
        };
        if (with_res && store_thread && (int)blockIdx.x < total_items) {
            pdl_wait();        // the residual is the result of an earlier kernel of the chain
            load_residual_dense(blockIdx.x, 0);
        }
        for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
            int tm = item, nt = 0;
            if (p.tiles_n > 1) { tm = item / p.tiles_n; nt = item - tm * p.tiles_n; }
            int n, p0, q0;
            tile_origin(p, tm, n, p0, q0);
            const int k0 = nt * p.FT;
            const int rows_valid = p.P - p0;                 // tile rows below this are real image rows
            // first pooled pixel of the tile (2x2 pool: full-width tiles from an even row)
            __nv_bfloat16 *ytile = p.pool == 1 ? p.y + ((size_t)n * (p.P >> 1) + (p0 >> 1)) * (p.Q >> 1) * p.k_pad : nullptr;
            ok = __all_sync(0xffffffffu, mbar_wait(tfull(acc), acc_phase, abort_flag, p.status, false));
            if (!ok) break;
            tc_fence_after();
            const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * p.MT * p.FT);
            if constexpr (DENSE) {
                // Flat task with one filter tile: the tile's output is ONE contiguous range of y (slot-major, k_pad filters
                // per slot).  With an odd number of 16-byte pieces per slot it is staged in exactly that layout (the pieces
                // of eight neighbouring slots fall in distinct banks) and leaves by a single bulk copy; a residual arrives
                // the same way.  With an even number the staged slots are one piece longer, and the tile moves by a tiled
                // copy whose box is that one piece wider than the tensor: the piece outside is not written (read as zeros).
                const uint32_t b = group_counter & 1u;
                uint8_t *buf = smem + (staging0 - base) + b * stage_buf_bytes;
                const uint32_t pitch = (uint32_t)p.dense_pitch;
                if (with_res) {
                    ok = __all_sync(0xffffffffu, mbar_wait(res_full(b), (group_counter >> 1) & 1u, abort_flag, p.status, false));
                    if (!ok) break;
                }
                for (int g = 0; g < groups; ++g) {
                    const int ch = g * 64 + half * 16;           // this warp's 16 filters of the group (16 epilogue warps)
                    if (ch >= p.k_pad) continue;
                    for (int mb = 0; mb < p.MT; ++mb) {
                        uint8_t *row = buf + (uint32_t)(mb * 128 + trow) * pitch;
                        uint32_t v[16];
                        tmem_ld16(t_row + (uint32_t)(mb * p.FT + ch), v);
                        bf16x8 rv[2];
                        if (with_res) {
#pragma unroll
                            for (int j = 0; j < 2; ++j)
                                if (ch + j * 8 < p.k_pad) rv[j] = *(const bf16x8 *)(row + (ch + j * 8) * 2);
                        }
                        tmem_ld_wait();
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            const int c = ch + q * 8;
                            if (c < p.k_pad) {
                                float f[8];
                                const float4 b0 = *(const float4 *)(bias_src + c);
                                const float4 b1 = *(const float4 *)(bias_src + c + 4);
                                const float bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
                                for (int j = 0; j < 8; ++j) f[j] = __uint_as_float(v[q * 8 + j]) + bb[j];
                                if (with_res) {
                                    float rf[8];
                                    unpack8(rv[q], rf);
#pragma unroll
                                    for (int j = 0; j < 8; ++j) f[j] += rf[j];
                                }
#pragma unroll
                                for (int j = 0; j < 8; ++j) f[j] = fminf(fmaxf(f[j], act_lo), act_hi);
                                *(bf16x8 *)(row + c * 2) = pack8(f);
                            }
                        }
                    }
                }
                // every warp has read what it needs of the accumulator (a warp without filters in the last group too)
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(tempty(acc));
                fence_async_smem();
                // the other buffer, written next, was last read by the previous tile's store
                if (store_thread) tma_store_wait_read<0>();
                ok = epi_sync();
                if (!ok) break;
                if (store_thread) {
                    const int rows = min(p.TW, p.Q - q0);
                    if (dense_tiled) tma_store_4d(&tm_y, staging0 + b * stage_buf_bytes, 0, q0, 0, 0);
                    else bulk_store(p.y + (size_t)q0 * p.k_pad, staging0 + b * stage_buf_bytes, (uint32_t)rows * pitch);
                    tma_store_commit();
                    if (with_res && item + (int)gridDim.x < total_items) load_residual_dense(item + gridDim.x, group_counter + 1);
                }
                ++group_counter;
            } else {
            for (int g = 0; g < groups && ok; ++g) {
                const uint32_t boff = (p.staging_bufs == 2 ? (group_counter & 1u) : 0u) * stage_buf_bytes;
                uint8_t *buf = smem + (staging0 - base) + boff;
                const int ch = g * 64 + half * 32;           // this warp's 32 filters of the group
                if constexpr (SPLIT) {
                    // the buffer's previous contents (two groups ago) must have been pooled
                    ok = __all_sync(0xffffffffu, mbar_wait(sempty(group_counter & 1u), ((group_counter >> 1) & 1u) ^ 1u, abort_flag, p.status, false));
                    if (!ok) break;
                }
                // Units of 16 filters of one accumulator block: (block 0, first 16), (block 0, second 16), (block 1, ...).
                // The tensor-memory load of unit u + 1 is in flight while unit u is turned into bf16 and staged, so that
                // only the first load's latency is exposed; two register buffers alternate.
                const bool u_ok[4] = {ch < p.FT, ch + 16 < p.FT, p.MT == 2 && ch < p.FT, p.MT == 2 && ch + 16 < p.FT};
                auto unit_addr = [&](int u) { return t_row + (uint32_t)((u >> 1) * p.FT + ch + (u & 1) * 16); };
                auto stage_unit = [&](int u, const uint32_t *v) {
                    const int c0 = ch + (u & 1) * 16;
                    float f[16];
                    if (bias_const) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) f[j] = __uint_as_float(v[j]) + bias_r[(u & 1) * 16 + j];
                    } else {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const float4 b4 = *(const float4 *)(bias_src + k0 + c0 + q * 4);
                            f[q * 4 + 0] = __uint_as_float(v[q * 4 + 0]) + b4.x;
                            f[q * 4 + 1] = __uint_as_float(v[q * 4 + 1]) + b4.y;
                            f[q * 4 + 2] = __uint_as_float(v[q * 4 + 2]) + b4.z;
                            f[q * 4 + 3] = __uint_as_float(v[q * 4 + 3]) + b4.w;
                        }
                    }
                    if (p.act == CPRUNE_ACT_RELU) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) f[j] = fmaxf(f[j], 0.f);
                    } else if (p.act == CPRUNE_ACT_RELU6) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) f[j] = fminf(fmaxf(f[j], 0.f), 6.f);
                    }
                    uint8_t *blk = buf + (u >> 1) * PK_BLOCK_BYTES;
                    *(bf16x8 *)(blk + sub_off(trow, half * 4 + (u & 1) * 2)) = pack8(f);
                    *(bf16x8 *)(blk + sub_off(trow, half * 4 + (u & 1) * 2 + 1)) = pack8(f + 8);
                };
                {
                    uint32_t va[16], vb[16];
                    if (u_ok[0]) tmem_ld16(unit_addr(0), va);
                    tmem_ld_wait();
                    if (u_ok[1]) tmem_ld16(unit_addr(1), vb);
                    if (u_ok[0]) stage_unit(0, va);
                    tmem_ld_wait();
                    if (u_ok[2]) tmem_ld16(unit_addr(2), va);
                    if (u_ok[1]) stage_unit(1, vb);
                    tmem_ld_wait();
                    if (u_ok[3]) tmem_ld16(unit_addr(3), vb);
                    if (u_ok[2]) stage_unit(2, va);
                    tmem_ld_wait();
                    if (g == groups - 1) {     // accumulator fully read: hand it back
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(tempty(acc));
                    }
                    if (u_ok[3]) stage_unit(3, vb);
                }
                if constexpr (SPLIT) {
                    // hand the staged group to the pooling warps and go on with the next one
                    __syncwarp();
                    if (lane == 0) mbar_arrive(sfull(group_counter & 1u));
                    ++group_counter;
                    continue;
                }
                if (!p.pool) {
                    // one TMA store per group: the staged slots are TH rows of Wp pixels; the tensor map's box has
                    // that shape, and the wrap-around columns (j >= Q), rows below the image and filters beyond
                    // k_pad fall outside the tensor, where a store writes nothing
                    fence_async_smem();
                    // the buffer written next (the other one) was last read by the previous group's store
                    if (p.staging_bufs == 2 && store_thread) tma_store_wait_read<0>();
                    ok = epi_sync();
                    if (!ok) break;
                    if (store_thread) {
                        if (k0 + g * 64 < p.k_pad) tma_store_4d(&tm_y, staging0 + boff, k0 + g * 64, q0, p0, n);
                        tma_store_commit();
                        if (p.staging_bufs == 1) tma_store_wait_read<0>();
                    }
                    if (p.staging_bufs == 1) {
                        ok = epi_sync();
                        if (!ok) break;
                    }
                    ++group_counter;
                    continue;
                }
                ok = epi_sync();
                if (!ok) break;
                // copy-out: eight threads per output pixel, 16 bytes each
                const int kg = k0 + g * 64;
                auto staged = [&](int sl, int chunk) { return *(const uint4 *)(buf + (sl >> 7) * PK_BLOCK_BYTES + sub_off(sl & 127, chunk)); };
                if (p.pool == 1) {
                    for (int e = etid; e < n_entries * 8; e += 256) {
                        const int2 l = lut[e >> 3];
                        const int chunk = e & 7;
                        if (l.x >= 0 && (l.x >> 16) < rows_valid && g * 64 + chunk * 8 < p.FT && kg + chunk * 8 < p.k_pad) {
                            const int slot = l.x & 0xffff;
                            uint4 val = bf16x8_max(staged(slot, chunk), staged(slot + 1, chunk));
                            val = bf16x8_max(val, bf16x8_max(staged(slot + p.Wp, chunk), staged(slot + p.Wp + 1, chunk)));
                            *(uint4 *)(ytile + l.y + kg + chunk * 8) = val;
                        }
                    }
                } else {
                    // 3x3 stride-2 windows: the tile computed conv rows p0 .. p0 + TH - 1 (p0 odd or -1) and holds the
                    // windows of (TH - 1) / 2 x (TW - 1) / 2 pooled pixels.  All nine slots of a window are inside the
                    // staged tile, so they are loaded unconditionally; conv pixels outside the image are replaced by
                    // -inf (they never win).
                    const int pr0 = (p0 + 1) >> 1, pc0 = (q0 + 1) >> 1;
                    const uint4 ninf = make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
                    // after ReLU / ReLU6 all values are >= 0: pixels outside the image can be replaced by 0 (every
                    // window holds a real pixel) and the maximum taken on the bit patterns
                    const uint4 fill = clamp_lo ? make_uint4(0u, 0u, 0u, 0u) : ninf;
#pragma unroll
                    for (int it = 0; it < 2; ++it) {
                        const int e = etid + it * 256;
                        const int chunk = e & 7;
                        const int pr = pr0 + win_pi[it], pc = pc0 + win_pj[it];
                        if (e < n_entries * 8 && pr < p.out_h && pc < p.out_w && g * 64 + chunk * 8 < p.FT && kg + chunk * 8 < p.k_pad) {
                            const int r0 = p0 + 2 * win_pi[it], c0 = q0 + 2 * win_pj[it];
                            // bit d of a mask: window row / column d lies inside the image
                            const uint32_t rmask = (r0 >= 0 ? 1u : 0u) | 2u | (r0 + 2 < p.P ? 4u : 0u);
                            const uint32_t cmask = (c0 >= 0 ? 1u : 0u) | 2u | (c0 + 2 < p.Q ? 4u : 0u);
                            uint4 w[9];
#pragma unroll
                            for (int k = 0; k < 9; ++k) {
                                const uint4 t = *(const uint4 *)(buf + win_off[it][k]);
                                w[k] = ((rmask >> (k / 3)) & (cmask >> (k % 3)) & 1u) ? t : fill;
                            }
                            uint4 m;
                            if (clamp_lo) {
                                const uint4 a0 = bf16x8_max_nonneg(bf16x8_max_nonneg(w[0], w[1]), bf16x8_max_nonneg(w[2], w[3]));
                                const uint4 a1 = bf16x8_max_nonneg(bf16x8_max_nonneg(w[4], w[5]), bf16x8_max_nonneg(w[6], w[7]));
                                m = bf16x8_max_nonneg(bf16x8_max_nonneg(a0, a1), w[8]);
                            } else {
                                const uint4 a0 = bf16x8_max(bf16x8_max(w[0], w[1]), bf16x8_max(w[2], w[3]));
                                const uint4 a1 = bf16x8_max(bf16x8_max(w[4], w[5]), bf16x8_max(w[6], w[7]));
                                m = bf16x8_max(bf16x8_max(a0, a1), w[8]);
                            }
                            *(uint4 *)(p.y + (((size_t)n * p.out_h + pr) * p.out_w + pc) * p.k_pad + kg + chunk * 8) = m;
                        }
                    }
                }
                if (p.staging_bufs == 1) {
                    ok = epi_sync();
                    if (!ok) break;
                }
                ++group_counter;
            }
            }
            if (p.acc_bufs == 2) { if (++acc == 2) { acc = 0; acc_phase ^= 1u; } }
            else acc_phase ^= 1u;
        }
        if (store_thread) tma_store_wait_all();      // staged data must be read before the CTA's memory goes away
    }

    // ---------------------------------------------------------------------- teardown
    if (*abort_flag) {
        for (int i = 0; i < 200; ++i) __nanosleep(1000);   // let copies in flight land before the memory goes away
    }
    tc_fence_before();
    __syncthreads();
    if (warp == PK_MMA_WARP) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// ------------------------------------------------------------------------------------------ host

// Estimated cycles of one tile.  Per tcgen05.mma (M = 128, N = FT, K = 16) the tensor pipe needs FT / 2 cycles
// and the operand reads (128 + FT) * 32 bytes of the 128 bytes per clock that shared memory delivers; the TMA
// writes of filters and patches share that port (measured on B200).
static double tile_cycles(int MT, int FT, int RS, int cblks, int ksteps_last, int row_bytes, int Wp, int TH, int R, bool resident,
                          int acc_bufs) {
    double total = 0;
    for (int cb = 0; cb < cblks; ++cb) {
        const int nk = cb == cblks - 1 ? ksteps_last : 4;
        const double tensor = MT * nk * (FT / 2.0);
        const double smem = (MT * nk * (128.0 + FT) * 32.0 + (resident ? 0.0 : FT * (double)row_bytes)) / 128.0;
        total += RS * (tensor > smem ? tensor : smem) + Wp * (TH + R - 1) * row_bytes / 128.0;
    }
    const double epilogue = MT * ((FT + 63) / 64) * 1200.0;
    return total + (acc_bufs == 2 ? (epilogue > total ? epilogue - total : 0.0) : epilogue) + 1500.0;
}

// What the kernel sees.  Wide tasks (c_pad >= 16, stride 1): the task itself, 64 channels per shared-memory row.
// Stems with C * stride^2 <= 16 (stride 1 or 2): the input is first regrouped into 16-channel pixels, one per
// stride x stride block of input pixels (channel (dy * stride + dx) * C + c), with the zero columns of the padding
// written out.  Up to four consecutive regrouped pixels (the Se filter columns, 32 bytes each) are then read as
// ONE 128-byte shared-memory row through a tensor map whose pixel stride is 32 bytes, so that the task becomes a
// stride-1 task with Re x 1 taps of Se * 16 channels and no wrap-around slots.  (Rows of 32 bytes would work too,
// but the MMA's operand reads then cost a full shared-memory cycle per row: measured four times slower.)
struct PatchGeometry {
    int stem, sf, Re, Se, pad_lo, He, We, WP, cblks, ksteps_last, Wp, kR, kS, pad_w;
    // the tensors as the kernel addresses them: images x rows x columns of the input (wide tasks) and of the conv output
    // and the stored output.  A 1x1 stride-1 task is a plain matrix product: its pixels are viewed as ONE row of
    // N*H*W columns, so that tiles are runs of 128 or 256 pixels with nothing wasted (flat = 1).
    int flat, vN, vH, vW, vP, vQ, vOH, vOW;
};

static bool patch_geometry(const cprune_plan_info &i, PatchGeometry *g) {
    if (i.groups != 1) return false;
    g->flat = 0; g->vN = i.N; g->vH = i.H; g->vW = i.W; g->vP = i.P; g->vQ = i.Q; g->vOH = i.out_h; g->vOW = i.out_w;
    if (i.c_pad >= 16 && i.stride == 1 && i.R == 1 && i.S == 1 && i.pad == 0) {
        const long long M = (long long)i.N * i.H * i.W;
        if (M > 0x7fffffffLL) return false;
        g->flat = 1; g->vN = 1; g->vH = 1; g->vW = (int)M; g->vP = 1; g->vQ = (int)M; g->vOH = 1; g->vOW = (int)M;
        g->stem = 0; g->sf = 1; g->Re = 1; g->Se = 1; g->pad_lo = 0; g->He = 1; g->We = (int)M; g->WP = (int)M;
        g->cblks = (i.c_pad + 63) / 64;
        g->ksteps_last = (i.c_pad - (g->cblks - 1) * 64 + 15) / 16;
        g->Wp = 128;                           // per tile: set by the planner (128 or 256 pixels)
        g->kR = 1; g->kS = 1; g->pad_w = 0;
        return true;
    } else if (i.c_pad >= 16 && i.stride == 1) {
        if (i.R * i.S <= 1 || i.R > 7 || i.S > 7) return false;
        g->stem = 0; g->sf = 1; g->Re = i.R; g->Se = i.S; g->pad_lo = i.pad; g->He = i.H; g->We = i.W; g->WP = i.W;
        g->cblks = (i.c_pad + 63) / 64;
        g->ksteps_last = (i.c_pad - (g->cblks - 1) * 64 + 15) / 16;
        g->Wp = i.Q + i.S - 1;
        g->kR = i.R; g->kS = i.S; g->pad_w = i.pad;
        if (g->Wp < g->We + g->pad_lo) return false;
    } else if (i.c_pad == 8 && i.stride <= 2 && i.C * i.stride * i.stride <= 16 && i.R * i.S > 1 && i.R <= 8 && i.S <= 8) {
        const int sf = i.stride;
        if ((i.H % sf) || (i.W % sf)) return false;
        if ((size_t)4 * sf * i.W * 16 > 48 * 1024) return false;   // the regrouping pass stages 4 * sf input rows in shared memory
        if (i.R - 1 - i.pad < 0 || i.S - 1 - i.pad < 0) return false;
        g->stem = 1; g->sf = sf;
        g->pad_lo = sf == 1 ? i.pad : (i.pad + 1) / 2;
        g->Re = sf == 1 ? i.R : (i.R - 1 - i.pad) / 2 + g->pad_lo + 1;
        g->Se = sf == 1 ? i.S : (i.S - 1 - i.pad) / 2 + g->pad_lo + 1;
        if (g->Se > 4) return false;
        g->He = i.H / sf; g->We = i.W / sf;
        g->WP = i.Q + 3;                       // a row starting at the last output column still reads four pixels
        if (g->WP < g->We + g->pad_lo) return false;
        g->cblks = 1; g->ksteps_last = g->Se;
        g->Wp = i.Q;
        g->kR = g->Re; g->kS = 1; g->pad_w = 0;
    } else {
        return false;
    }
    if (g->Wp > 128) return false;
    if (i.P + g->Re - 1 < g->He + g->pad_lo) return false;
    return true;
}

// Decides whether the task runs on the patch kernel and with which tiling; fills plan->info tile fields.
cprune_status plan_conv_patch(cprune_plan *plan) {
    cprune_plan_info &i = plan->info;
    plan->patch = 0;
    plan->pre_bytes = 0;
    PatchGeometry g;
    if (!patch_geometry(i, &g)) return CPRUNE_ERR_UNSUPPORTED;
    const bool pool = plan->opts.pool == CPRUNE_POOL_MAX2X2;
    const bool pool3 = plan->opts.pool == CPRUNE_POOL_MAX3X3S2;
    if (pool && (plan->opts.residual || (i.P & 1) || (i.Q & 1))) return CPRUNE_ERR_UNSUPPORTED;
    // the 3x3 pool needs tiles narrower than the image, which only tasks without wrap-around slots allow
    if (pool3 && (plan->opts.residual || g.kS != 1)) return CPRUNE_ERR_UNSUPPORTED;
    if (g.flat && (pool || pool3)) return CPRUNE_ERR_UNSUPPORTED;
    const int k16 = round_up(i.K, 16);
    const int cblks = g.cblks, ksteps_last = g.ksteps_last, RB = 128;
    const int RS = g.kR * g.kS;
    double best = 1e30;
    PatchTiling bt = {};
    for (int MT = 1; MT <= 2; ++MT) {
      // candidate tile shapes: whole-width rows; for the 3x3 pool (2 tpr + 1) x (2 tpc + 1) conv pixels around tpr x tpc pooled ones
      const int n_shapes = pool3 ? 32 * 32 : 1;
      for (int shape = 0; shape < n_shapes; ++shape) {
        int TH, TW = g.vQ, tiles_w = 1, step_h, step_w = g.vQ, org = 0, tiles_per_img, Wp = g.Wp;
        if (g.flat) {
            TH = 1; TW = 128 * MT; Wp = TW; step_h = 1; step_w = TW;
            tiles_w = (g.vQ + TW - 1) / TW;
            tiles_per_img = tiles_w;
        } else if (pool3) {
            const int tpr = shape / 32 + 1, tpc = shape % 32 + 1;
            if (tpr > i.out_h || tpc > i.out_w) continue;
            TH = 2 * tpr + 1; TW = 2 * tpc + 1;
            if (TH * TW > 128 * MT) continue;
            Wp = TW;
            step_h = 2 * tpr; step_w = 2 * tpc; org = -1;
            tiles_w = (i.out_w + tpc - 1) / tpc;
            tiles_per_img = ((i.out_h + tpr - 1) / tpr) * tiles_w;
        } else {
            TH = (128 * MT) / Wp;
            if (TH > i.P) TH = i.P;
            if (pool) TH &= ~1;
            if (TH < 1) continue;
            step_h = TH;
            tiles_per_img = (i.P + TH - 1) / TH;
        }
        for (int tiles_n = 1; tiles_n <= 8; ++tiles_n) {
            // with several filter tiles every tile ends on a 64-filter boundary: the stores are 64 filters wide and
            // only the tensor's own edge clips them
            const int FT = round_up((k16 + tiles_n - 1) / tiles_n, tiles_n > 1 ? 64 : 16);
            if (FT > 256 || MT * FT > 512) continue;
            if ((k16 + FT - 1) / FT != tiles_n) continue;
            const int acc_bufs = 2 * MT * FT <= 512 ? 2 : 1;
            const int patch_bytes = round_up((128 * MT + (g.kR - 1) * Wp + g.kS - 1) * RB, 1024);
            if (patch_bytes < Wp * (TH + g.kR - 1) * RB) continue;
            // patch ring depth: two stages; up to four when the task has that many channel blocks and the patches are
            // small (1x1 tasks), because each load's latency is otherwise exposed
            // (flat tasks: a tile is little work, and a patch load's latency under a stream of output writes is several
            // tiles long, so the ring is as deep as fits)
            int ps_max = 2;
            if (cblks > 2 && patch_bytes <= 32 * 1024) ps_max = cblks < PK_MAX_PATCH_STAGES ? cblks : PK_MAX_PATCH_STAGES;
            if (g.flat || g.stem) ps_max = PK_MAX_PATCH_STAGES;     // (stems: a tile is a few MMAs, shorter than a load's latency)
            // A residual travels through the patch ring too (64 filters per stage).  A deeper ring, which would let the
            // next tile's first patch be fetched while the residual blocks are still in use, was measured against the
            // shallow one with the shared memory spent on resident filters / more filter stages instead: the shallow ring
            // won on every ResNet-18 shape (26.5 vs 27.8 us, 21.1 vs 22.5 us, 21.9 vs 21.7 us).
            const int res_blocks_plan = plan->opts.residual ? (FT + 63) / 64 : 0;
          for (int pstages = ps_max; pstages >= 2; --pstages) {
            const int dense_pitch = ((((i.k_pad >> 3) & 1) || i.k_pad == 16) ? i.k_pad : i.k_pad + 8) * 2;
            const int dense_bytes = round_up(128 * MT * dense_pitch, 1024);
            const int dense = g.flat && tiles_n == 1 && dense_pitch <= 512 && dense_bytes <= 48 * 1024 &&
                              (dense_pitch == i.k_pad * 2 || !plan->opts.residual);
            // a residual is added on the tensor core (identity operand in shared memory), except with dense staging,
            // where it arrives in the staging buffer
            const int ident_bytes = (plan->opts.residual && !dense) ? PK_IDENT_BYTES : 0;
            const int fixed = 1024 + pstages * patch_bytes + PK_CTRL_BYTES + ident_bytes;
            const int budget = 227 * 1024 - fixed;
            const int sb_max = 2, sb_min = 1;
            const int w_stage = round_up(FT * RB, 1024);
            // flat tasks with one filter tile stage the tile as it lies in memory (k_pad filters per pixel) when that fits,
            // with the pixel pitch made an odd number of 16-byte pieces (no bank conflicts between neighbouring pixels;
            // 32-byte pixels conflict two-way and still gain, measured)
            const int stage_bytes = dense ? dense_bytes : MT * PK_BLOCK_BYTES;
            int staging_bufs = sb_max, wstages = 0, resident = 0;
            // resident filters when the whole set of this filter tile fits
            const int sb_res_min = sb_min;
            if (tiles_n == 1 && RS * cblks <= PK_MAX_WSTAGES) {
                for (int sb = sb_max; sb >= sb_res_min && !resident; --sb)
                    if (RS * cblks * w_stage + sb * stage_bytes <= budget) { resident = 1; staging_bufs = sb; wstages = RS * cblks; }
            }
            if (!resident) {
                staging_bufs = sb_max;
                wstages = (budget - staging_bufs * stage_bytes) / w_stage;
                if (wstages < 3 && sb_min < sb_max) {
                    staging_bufs = sb_min;
                    wstages = (budget - staging_bufs * stage_bytes) / w_stage;
                }
                if (wstages < 3) continue;
                if (wstages > 8) wstages = 8;
            }
            if (dense && staging_bufs != 2) continue;
            // the fused 3x3 pool runs on its own warps only beside two staging buffers, which is worth more than a deeper ring
            if (pool3 && staging_bufs != 2 && pstages > 2) continue;
            const long long tiles = (long long)g.vN * tiles_per_img * tiles_n;
            const double waves = (double)((tiles + 147) / 148);
            double tile = tile_cycles(MT, FT, RS, cblks, ksteps_last, RB, Wp, TH, g.kR, resident != 0, acc_bufs);
            if (res_blocks_plan && !dense) tile += res_blocks_plan * (MT * 4 * 48.0 + TH * Wp);   // residual MMAs and their loads
            double t = waves * tile;
            if (resident) t += RS * cblks * FT;    // one-time filter load
            if (t < best) {
                best = t;
                bt = {MT, TH, FT, tiles_n, tiles_per_img, wstages, resident, acc_bufs, staging_bufs, patch_bytes, TW, tiles_w, step_h, step_w, org, pstages, dense, stage_bytes, dense_pitch};
            }
            break;      // the deepest ring that fits
          }
        }
      }
    }
    if (best >= 1e30) return CPRUNE_ERR_UNSUPPORTED;
    // share of accumulator rows that hold real pixels; below one half the im2col kernel is the better choice
    const double fill = (double)g.vP * g.vQ / ((double)bt.tiles_per_img * 128 * bt.MT);
    if (fill < 0.5) return CPRUNE_ERR_UNSUPPORTED;
    // too few tiles for the SMs: the im2col kernel can split the reduction over more CTAs
    if ((long long)g.vN * bt.tiles_per_img * bt.tiles_n < 64) return CPRUNE_ERR_UNSUPPORTED;
    plan->patch = 1;
    plan->pt = bt;
    plan->narrow = g.stem;
    plan->orient = 0;
    plan->small_c = 0;
    plan->s_packed = i.S;
    plan->splits = 1;
    plan->ipp = 0;
    plan->partial_bytes = 0;
    plan->pre_bytes = g.stem ? ((size_t)i.N * g.He * g.WP * 32 + 255) / 256 * 256 : 0;
    plan->fused_pool = (pool || pool3) ? 1 : 0;
    i.tile_m = 128 * bt.MT;
    i.tile_n = bt.FT;
    i.tile_k = 64;
    i.stages = bt.wstages;
    i.tiles_m = g.vN * bt.tiles_per_img;
    i.tiles_n = bt.tiles_n;
    i.k_alloc = bt.tiles_n * bt.FT;
    const int ksteps = (cblks - 1) * 4 + ksteps_last;
    i.padded_flops = 2.0 * (double)i.tiles_m * i.tile_m * (double)i.k_alloc * RS * ksteps * 16.0;
    plan->smem_bytes = 1024 + bt.pstages * bt.patch_bytes + bt.wstages * round_up(bt.FT * RB, 1024) +
                       bt.staging_bufs * bt.stage_bytes + PK_CTRL_BYTES + ((plan->opts.residual && !bt.dense) ? PK_IDENT_BYTES : 0);
    plan->est_us = best / 1900.0 + 4.0;      // cycles at about 1.9 GHz plus launch, set-up and drain
    return CPRUNE_OK;
}

// Regroups an NHWC tensor with C channels per pixel (T = bf16 with 8 channel lanes in memory, or float32 with C) into
// 16-channel bf16 pixels, one per sf x sf block of input pixels, in rows of WP pixels of which the first pad_lo (and
// whatever follows the image) are zero:
//   out[n][h2][pad_lo + w2][(dy * sf + dx) * C + c] = x[n][sf * h2 + dy][sf * w2 + dx][c], other channels zero.
// Two threads per output pixel, eight channels (one 16-byte store) each.
constexpr int RG_ROWS = 4;     // regrouped rows per block

template <typename T>
__global__ void __launch_bounds__(256) regroup_kernel(const T *__restrict__ x, int H, int W, int C, int c_mem, int sf, int pad_lo, int WP,
                                                      uint4 *__restrict__ out) {
    pdl_trigger();
    pdl_wait();
    // one block per RG_ROWS regrouped rows of one image: their sf * RG_ROWS input rows are contiguous in memory and are
    // brought into shared memory with 16-byte loads first
    extern __shared__ __align__(16) unsigned char rg_smem[];
    __shared__ int src_off[16];            // regrouped channel -> offset within an sf x sf input block, or -1 (zero)
    T *srow = reinterpret_cast<T *>(rg_smem);
    const int H2 = H / sf, W2 = W / sf;
    const int blocks_per_img = (H2 + RG_ROWS - 1) / RG_ROWS;
    const int n = blockIdx.x / blocks_per_img;
    const int h2_0 = (blockIdx.x - n * blocks_per_img) * RG_ROWS;
    const int nrows = min(RG_ROWS, H2 - h2_0);
    const T *rows = x + ((size_t)n * H + (size_t)sf * h2_0) * W * c_mem;
    const int row_elems = sf * W * c_mem;                // input elements behind one regrouped row
    const int n_elems = nrows * row_elems;
    const size_t n_bytes = (size_t)n_elems * sizeof(T);
    if (threadIdx.x < 16) {
        const int ch = threadIdx.x, blk = ch / C, c = ch - blk * C;
        const int dy = blk / sf, dx = blk - dy * sf;
        src_off[ch] = blk < sf * sf ? (dy * W + dx) * c_mem + c : -1;
    }
    if (((reinterpret_cast<uintptr_t>(rows) | n_bytes) & 15) == 0) {
        const uint4 *src = reinterpret_cast<const uint4 *>(rows);
        uint4 *dst = reinterpret_cast<uint4 *>(rg_smem);
        const int n16 = (int)(n_bytes >> 4);
        // four loads in flight per thread: the block's latency is one round trip to memory, not one per 4 KB
        for (int i0 = threadIdx.x; i0 < n16; i0 += 4 * 256) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (i0 + u * 256 < n16) v[u] = __ldg(src + i0 + u * 256);
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (i0 + u * 256 < n16) dst[i0 + u * 256] = v[u];
        }
    } else {
        for (int i = threadIdx.x; i < n_elems; i += blockDim.x) srow[i] = rows[i];
    }
    __syncthreads();
    uint4 *orow = out + ((size_t)n * H2 + h2_0) * WP * 2;
    const int per_row = WP * 2;
    const int step = sf * c_mem;                         // input elements between neighbouring regrouped pixels
    for (int e = threadIdx.x; e < nrows * per_row; e += blockDim.x) {
        const int r = e / per_row, c = e - r * per_row;
        const int half = c & 1, w2 = (c >> 1) - pad_lo;
        float v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) v[k] = 0.f;
        if (w2 >= 0 && w2 < W2) {
            const T *in = srow + (size_t)r * row_elems + w2 * step;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int o = src_off[half * 8 + k];
                if (o >= 0) v[k] = (float)in[o];
            }
        }
        const bf16x8 q = pack8(v);
        orow[e] = *reinterpret_cast<const uint4 *>(&q);
    }
}

// Filters of a regrouped stem: out[k][re * Se + se][(dy * sf + dx) * C + c] = w[k][c][sf * re + dy - er][sf * se + dx - es]
// (zero where that tap does not exist), er = sf * pad_lo - pad.  Rows k >= K are zero.
__global__ void __launch_bounds__(256) pack_regrouped_kernel(const float *__restrict__ w, int K, int C, int R, int S, int sf, int Re,
                                                             int Se, int er, int es, int k_alloc, __nv_bfloat16 *__restrict__ out) {
    const size_t total = (size_t)k_alloc * Re * Se * 16;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
        const int ch = (int)(e % 16);
        size_t t = e / 16;
        const int se = (int)(t % Se); t /= Se;
        const int re = (int)(t % Re);
        const int k = (int)(t / Re);
        float v = 0.f;
        const int blk = ch / C, c = ch - blk * C;
        if (k < K && blk < sf * sf) {
            const int dy = blk / sf, dx = blk - dy * sf;
            const int r = sf * re + dy - er, s2 = sf * se + dx - es;
            if (r >= 0 && r < R && s2 >= 0 && s2 < S) v = w[(((size_t)k * C + c) * R + r) * S + s2];
        }
        out[e] = __float2bfloat16_rn(v);
    }
}

cprune_status pack_conv_patch(const cprune_plan *plan, const float *w, void *w_packed, cudaStream_t st) {
    const cprune_plan_info &i = plan->info;
    PatchGeometry g;
    if (!patch_geometry(i, &g) || !g.stem) return CPRUNE_ERR_INTERNAL;
    const size_t total = (size_t)i.k_alloc * g.Re * g.Se * 16;
    size_t blocks = (total + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    pack_regrouped_kernel<<<(unsigned)blocks, 256, 0, st>>>(w, i.K, i.C, i.R, i.S, g.sf, g.Re, g.Se, g.sf * g.pad_lo - i.pad,
                                                           g.sf * g.pad_lo - i.pad, i.k_alloc, (__nv_bfloat16 *)w_packed);
    CPRUNE_LAUNCH_CHECK("pack_regrouped_kernel");
    return CPRUNE_OK;
}

size_t packed_weight_bytes_patch(const cprune_plan *plan) {
    const cprune_plan_info &i = plan->info;
    PatchGeometry g;
    if (!patch_geometry(i, &g) || !g.stem) return 0;
    return (size_t)i.k_alloc * g.Re * g.Se * 32;
}

cprune_status regroup_stem_input(const cprune_plan *plan, const void *x, int x_is_f32, void *scratch, cudaStream_t st) {
    const cprune_plan_info &i = plan->info;
    PatchGeometry g;
    if (!patch_geometry(i, &g) || !g.stem || !x || !scratch) return CPRUNE_ERR_INVALID_ARG;
    const unsigned blocks = (unsigned)(i.N * ((g.He + RG_ROWS - 1) / RG_ROWS));
    const size_t row_bytes = (size_t)RG_ROWS * g.sf * i.W * (x_is_f32 ? (size_t)i.C * 4 : (size_t)i.c_pad * 2);
    if (row_bytes > 48 * 1024) return CPRUNE_ERR_UNSUPPORTED;     // planning keeps such images off this path
    if (x_is_f32)
        CPRUNE_CUDA_CHECK(launch_chained(regroup_kernel<float>, dim3(blocks), dim3(256), row_bytes, st, (const float *)x, i.H, i.W, i.C, i.C, g.sf, g.pad_lo,
                                         g.WP, (uint4 *)scratch));
    else
        CPRUNE_CUDA_CHECK(launch_chained(regroup_kernel<__nv_bfloat16>, dim3(blocks), dim3(256), row_bytes, st, (const __nv_bfloat16 *)x, i.H, i.W, i.C,
                                         i.c_pad, g.sf, g.pad_lo, g.WP, (uint4 *)scratch));
    return CPRUNE_OK;
}

cprune_status launch_conv_patch(cprune_plan *plan, const void *x, const void *w, const float *b, const void *res, void *y,
                                void *scratch, cudaStream_t st, bool input_regrouped) {
    const cprune_plan_info &i = plan->info;
    const PatchTiling &t = plan->pt;
    PatchGeometry g;
    if (!patch_geometry(i, &g)) return CPRUNE_ERR_INTERNAL;
    const int Wp = t.TW + g.kS - 1;    // patch row pitch: the tile's width plus the filter's
    const void *xe = x;        // the tensor the patch loads read
    if (g.stem) {
        if (!scratch) return CPRUNE_ERR_INVALID_ARG;
        if (!input_regrouped) {
            cprune_status rs = regroup_stem_input(plan, x, 0, scratch, st);
            if (rs != CPRUNE_OK) return rs;
        }
        xe = scratch;
    }
    CUtensorMap tm_x, tm_w, tm_y, tm_res;
    {
        std::lock_guard<std::mutex> lock(plan->mu);
        if (plan->map_x != xe) {
            if (g.stem) {
                // rows of 64 values = four consecutive regrouped pixels; start positions are one pixel (32 bytes) apart
                const unsigned long long dims[4] = {64, (unsigned long long)i.Q, (unsigned long long)g.He, (unsigned long long)i.N};
                const unsigned long long strides[3] = {32, (unsigned long long)g.WP * 32, (unsigned long long)g.He * g.WP * 32};
                const unsigned box[4] = {64, (unsigned)Wp, (unsigned)(t.TH + g.kR - 1), 1};
                cprune_status s = encode_tiled_bf16_swz(&plan->tm_a, xe, 4, dims, strides, box, 128, true);
                if (s != CPRUNE_OK) return s;
            } else {
                const unsigned long long dims[4] = {(unsigned long long)i.c_pad, (unsigned long long)g.vW, (unsigned long long)g.vH,
                                                    (unsigned long long)g.vN};
                const unsigned long long strides[3] = {(unsigned long long)i.c_pad * 2, (unsigned long long)g.vW * i.c_pad * 2,
                                                       (unsigned long long)g.vH * g.vW * i.c_pad * 2};
                const unsigned box[4] = {64, (unsigned)Wp, (unsigned)(t.TH + g.kR - 1), 1};
                cprune_status s = encode_tiled_bf16_swz(&plan->tm_a, xe, 4, dims, strides, box, 128, true);
                if (s != CPRUNE_OK) return s;
            }
            plan->map_x = xe;
        }
        if (plan->map_w != w) {
            // filters [k_alloc][taps][channels of a tap]; a stem's tap is a filter row: Se pixels of 16 channels
            const unsigned long long ctap = g.stem ? (unsigned long long)g.Se * 16 : (unsigned long long)i.c_pad;
            const unsigned long long taps = (unsigned long long)(g.kR * g.kS);
            const unsigned long long dims[3] = {ctap, taps, (unsigned long long)i.k_alloc};
            const unsigned long long strides[2] = {ctap * 2, taps * ctap * 2};
            const unsigned box[3] = {64, 1, (unsigned)t.FT};
            cprune_status s = encode_tiled_bf16_swz(&plan->tm_b, w, 3, dims, strides, box, 128, true);
            if (s != CPRUNE_OK) return s;
            plan->map_w = w;
        }
        if (plan->map_y != y) {
            // output [N][P][Q][k_pad]; a store is 64 filters x Wp pixels x TH rows (see the epilogue).  With a fused
            // pool the kernel stores by hand and the map is not used.
            const unsigned long long dims[4] = {(unsigned long long)i.k_pad, (unsigned long long)g.vOW, (unsigned long long)g.vOH,
                                                (unsigned long long)g.vN};
            const unsigned long long strides[3] = {(unsigned long long)i.k_pad * 2, (unsigned long long)g.vOW * i.k_pad * 2,
                                                   (unsigned long long)g.vOH * g.vOW * i.k_pad * 2};
            const bool dense_tiled = t.dense && t.dense_pitch != i.k_pad * 2;      // the whole staged tile, unswizzled
            const unsigned box[4] = {dense_tiled ? (unsigned)(t.dense_pitch / 2) : 64u, dense_tiled ? (unsigned)t.TW : (unsigned)Wp,
                                     dense_tiled ? 1u : (unsigned)t.TH, 1};
            cprune_status s = encode_tiled_bf16_swz(&plan->tm_y, y, 4, dims, strides, box, dense_tiled ? 0 : 128, false);
            if (s != CPRUNE_OK) return s;
            plan->map_y = y;
        }
        if (res && plan->map_res != res) {
            const unsigned long long dims[4] = {(unsigned long long)i.k_pad, (unsigned long long)g.vQ, (unsigned long long)g.vP,
                                                (unsigned long long)g.vN};
            const unsigned long long strides[3] = {(unsigned long long)i.k_pad * 2, (unsigned long long)g.vQ * i.k_pad * 2,
                                                   (unsigned long long)g.vP * g.vQ * i.k_pad * 2};
            const bool dense_tiled = t.dense && t.dense_pitch != i.k_pad * 2;
            const unsigned box[4] = {dense_tiled ? (unsigned)(t.dense_pitch / 2) : 64u, dense_tiled ? (unsigned)t.TW : (unsigned)Wp,
                                     dense_tiled ? 1u : (unsigned)t.TH, 1};
            cprune_status s = encode_tiled_bf16_swz(&plan->tm_res, res, 4, dims, strides, box, dense_tiled ? 0 : 128, true);
            if (s != CPRUNE_OK) return s;
            plan->map_res = res;
        }
        std::memcpy(&tm_x, &plan->tm_a, sizeof(CUtensorMap));
        std::memcpy(&tm_w, &plan->tm_b, sizeof(CUtensorMap));
        std::memcpy(&tm_y, &plan->tm_y, sizeof(CUtensorMap));
        std::memcpy(&tm_res, res ? &plan->tm_res : &plan->tm_y, sizeof(CUtensorMap));
    }
    // the shared-memory limit of a kernel is a per-device attribute
    static std::mutex attr_mu;
    static bool attr_set[64] = {false};
    {
        int dev = 0;
        CPRUNE_CUDA_CHECK(cudaGetDevice(&dev));
        if (dev < 0 || dev >= 64) return CPRUNE_ERR_UNSUPPORTED;
        std::lock_guard<std::mutex> lock(attr_mu);
        if (!attr_set[dev]) {
            CPRUNE_CUDA_CHECK(cudaFuncSetAttribute(conv_patch_kernel<PK_GENERAL>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            CPRUNE_CUDA_CHECK(cudaFuncSetAttribute(conv_patch_kernel<PK_DENSE>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            CPRUNE_CUDA_CHECK(cudaFuncSetAttribute(conv_patch_kernel<PK_POOL3>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            attr_set[dev] = true;
        }
    }
    PatchParams p;
    p.P = g.vP; p.Q = g.vQ; p.Wp = Wp; p.TH = t.TH; p.tiles_per_img = t.tiles_per_img;
    p.TW = t.TW; p.tiles_w = t.tiles_w; p.step_h = t.step_h; p.step_w = t.step_w; p.org = t.org;
    p.out_h = g.vOH; p.out_w = g.vOW;
    p.tiles_m = i.tiles_m; p.tiles_n = i.tiles_n; p.FT = t.FT; p.MT = t.MT; p.R = g.kR; p.S = g.kS; p.pad = g.pad_lo; p.pad_w = g.pad_w;
    p.cblks = g.cblks;
    p.ksteps_last = g.ksteps_last;
    p.k_pad = i.k_pad;
    p.act = plan->opts.activation;
    p.wstages = t.wstages; p.pstages = t.pstages; p.resident = t.resident; p.acc_bufs = t.acc_bufs; p.staging_bufs = t.staging_bufs;
    p.pool = plan->fused_pool ? plan->opts.pool : 0;
    p.patch_bytes = t.patch_bytes;
    p.patch_box_bytes = Wp * (t.TH + g.kR - 1) * 128;
    p.rb16 = 8;
    p.dense = t.dense; p.stage_bytes = t.stage_bytes; p.dense_pitch = t.dense_pitch;
    p.w_stage_bytes = t.FT * 128;
    p.bias = b;
    // dense staging takes the residual through the staging buffer; everywhere else the MMA warps add it
    p.res = t.dense ? (const __nv_bfloat16 *)res : nullptr;
    p.res_blocks = (res && !t.dense) ? (t.FT + 63) / 64 : 0;
    p.y = (__nv_bfloat16 *)y;
    p.status = device_status_word();
    if (!p.status) return cuda_fail(cudaGetLastError(), "status word");
    const int total = i.tiles_m * i.tiles_n;
    if (total == 0) return CPRUNE_OK;
    int sms = 148, dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
    const int grid = total < sms ? total : sms;
    // a fused 3x3 pool with two staging buffers: the instantiation with separate pooling warps
    const bool split_pool = p.pool == CPRUNE_POOL_MAX3X3S2 && t.staging_bufs == 2 && !res && !(plan->opts.flags & CPRUNE_FLAG_POOL_ON_EPILOGUE_WARPS);
    if (t.dense)
        CPRUNE_CUDA_CHECK(launch_chained(conv_patch_kernel<PK_DENSE>, dim3(grid), dim3(pk_threads(PK_DENSE)), (size_t)plan->smem_bytes, st, tm_x, tm_w, tm_y, tm_res, p));
    else if (split_pool)
        CPRUNE_CUDA_CHECK(launch_chained(conv_patch_kernel<PK_POOL3>, dim3(grid), dim3(pk_threads(PK_POOL3)), (size_t)plan->smem_bytes, st, tm_x, tm_w, tm_y, tm_res, p));
    else
        CPRUNE_CUDA_CHECK(launch_chained(conv_patch_kernel<PK_GENERAL>, dim3(grid), dim3(pk_threads(PK_GENERAL)), (size_t)plan->smem_bytes, st, tm_x, tm_w, tm_y, tm_res, p));
    return CPRUNE_OK;
}

}  // namespace cprune
