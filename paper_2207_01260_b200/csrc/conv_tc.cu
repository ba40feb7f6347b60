// Dense conv task as an implicit GEMM on the sm_100a tensor cores (paper Sec. 3.4: a task is
// Conv2d + folded BatchNorm + activation; Sec. 3.5: the filter count K is whatever pruning left).
//
//   D[pixel][k] = sum over (r, s, c) of  X[pixel shifted by tap (r,s)][c] * Wt[k][r][s][c]
//   GEMM-M = N*P*Q output pixels,  GEMM-N = K filters,  GEMM-K = R*S*C
//
// One persistent CTA per SM, 10 warps, three roles (measured: one producer warp is enough for this
// kernel, which is bound by shared-memory bandwidth):
//   warp 0      producer: per (tap, 64-channel block) one im2col-mode TMA load of PT pixels x 64
//               channels of the activation tensor (zero fill for the padding border and for
//               channels beyond c_pad) and one tiled TMA load of FT filters x 64 channels, both
//               into 128-byte-swizzled shared memory, completion on an mbarrier;
//   warp 1      one elected lane issues tcgen05.mma (K = 16 per instruction, bf16 x bf16 ->
//               float32) with the accumulator in tensor memory; two accumulator buffers so
//               that the epilogue of one tile overlaps the main loop of the next;
//   warps 2..9  epilogue: tcgen05.ld the accumulator, bias (+ residual), activation, bf16,
//               write 64-filter-wide sub-tiles into swizzled shared memory, TMA-store them to
//               the NHWC output (the store clips rows beyond the last pixel and filters beyond
//               k_pad by itself).
// An MMA instruction costs about the same for any N up to 256, so the plan picks the orientation
// that keeps N large:
//   ORIENT_PIX  (K > 128): MMA-M = 128 pixels,  MMA-N = BN filters (multiple of 16, <= 256);
//   ORIENT_FILT (K <= 128): MMA-M = 128 filter rows (zero rows above K), MMA-N = 256 pixels.
// Odd channel counts: C is padded to a multiple of 8 in memory and the last channel block issues
// only ceil(remaining/16) MMAs.  Every wait is bounded: when a limit expires the CTA raises
// STATUS_TIMEOUT in the device status word, all roles leave their loops, tensor memory is
// released and the kernel returns.
#include <cuda.h>

#include <cstdlib>
#include <cstring>
#include <mutex>

#include "common.cuh"
#include "plan.h"
#include "sm100_ptx.cuh"

namespace cprune {

constexpr int N_PRODUCERS = 1;     // TMA-issuing warps: pipeline stage i is filled by warp i % N_PRODUCERS
constexpr int MMA_WARP = N_PRODUCERS;
constexpr int FIRST_EPI_WARP = N_PRODUCERS + 1;
constexpr int TC_THREADS = (N_PRODUCERS + 1 + 8) * 32;    // producer warps, MMA warp, eight epilogue warps
constexpr int BK = 64;             // channels per stage: 64 bf16 = one 128-byte swizzle row
constexpr int TMEM_COLS = 512;
constexpr int ACC_STRIDE = 256;    // column offset of the second accumulator buffer
constexpr int MAX_STAGES = 8;
constexpr int ORIENT_PIX = 0, ORIENT_FILT = 1;
constexpr int SUB = 64;            // filters per staged sub-tile (128-byte rows, 128-byte swizzle)
constexpr int CTRL_BYTES = 2048;   // barriers, flags, bias vector
constexpr int GROUP_BYTES = 16384; // one staging buffer (see the kernel)
constexpr int POOL_SUB_BYTES = 16 * 128;   // pooled sub-tile of the filter-major orientation: 16 pixels x 64 filters

struct TcParams {
    long long M;
    int P, Q, stride, pad, R, S;
    int cblks;         // ceil(c_pad / 64)
    int ksteps_last;   // 16-channel MMA steps in the last channel block
    int PT, FT;        // pixels and filters per tile
    int tiles_m, tiles_n, k_pad, stages, act;
    int small_c;       // c_pad == 8 (3-channel stems): 1 = a 64-wide K block is 8 taps x 8 channels;
                       // 2 = stride-2 stems read as pixel pairs: 4 pair-taps x 16 channels per K block
    int pair_taps;     // small_c == 2: pair-taps per filter row, (S + 1) / 2
    int iters;         // pipeline stages per tile (K blocks, plus residual blocks)
    int res_iters;     // ORIENT_FILT with a residual: trailing stages that add it on the tensor core
    int pool;          // 1: 2x2 stride-2 max-pool fused into the epilogue (tm_y then maps the pooled output)
    int splits;        // split-K: CTAs that share one output tile, each a slice of the K blocks
    int ipp;           // K blocks per slice
    float *partial;    // [splits][M][k_alloc] when splits > 1
    const float *bias;
    const __nv_bfloat16 *res;
    int *status;
};
// Measured on B200: with kernel parameters beyond 768 bytes (five 128-byte tensor maps + this struct) tasks with
// many short tiles ran almost twice as slow; the struct therefore has to stay within 128 bytes.
static_assert(sizeof(TcParams) <= 128, "conv_tc_kernel parameters must stay within 768 bytes");

// 2x2 stride-2 max-pool of NPX consecutive pixels (whole row pairs of Q pixels, Q a power of two) held by
// one thread for one filter: NPX / 4 pooled values, written to rows t0.. of a staged sub-tile.
template <int Q, int NPX>
__device__ __forceinline__ void store_pooled(const float *f, uint8_t *dst, int chunk, int t0) {
#pragma unroll
    for (int t = 0; t < NPX / 4; ++t) {
        const int rp = t / (Q / 2), cq = t % (Q / 2);
        const int b = rp * 2 * Q + 2 * cq;
        const float m = fmaxf(fmaxf(f[b], f[b + 1]), fmaxf(f[b + Q], f[b + Q + 1]));
        *(__nv_bfloat16 *)(dst + sub_off(t0 + t, chunk)) = __float2bfloat16_rn(m);
    }
}

// ---------------------------------------------------------------------------------------- kernel

template <int ORIENT, int POOL>
__global__ void __launch_bounds__(TC_THREADS, 1)
conv_tc_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
               const __grid_constant__ CUtensorMap tm_y, const __grid_constant__ CUtensorMap tm_res,
               const __grid_constant__ CUtensorMap tm_id, const TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    pdl_trigger();
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;          // swizzled tiles need 1024-byte alignment
    uint8_t *smem = smem_raw + (base - raw);
    const int x_bytes = p.PT * BK * 2;                     // pixel operand of one stage
    const int stage_bytes = x_bytes + p.FT * BK * 2;
    // staging buffers, each one group of sub-tiles [rows][64 filters] bf16:
    //   ORIENT_PIX:  128 pixels x 64 filters  = 1 sub-tile of 16 KB
    //   ORIENT_FILT:  64 pixels x 128 filters = 2 sub-tiles of 8 KB
    constexpr int GROUP_ROWS = ORIENT == ORIENT_PIX ? 128 : 64;
    constexpr int SUB_BYTES = GROUP_ROWS * SUB * 2;
    const uint32_t staging0 = base + (uint32_t)p.stages * stage_bytes;
    const uint32_t ctrl0 = staging0 + 2u * GROUP_BYTES;
    uint8_t *ctrl = smem + (ctrl0 - base);
    // barrier slots (8 bytes each): full[8], empty[8], tfull[2], tempty[2], epi[1]
    auto full_bar = [&](int s) { return ctrl0 + 8u * s; };
    auto empty_bar = [&](int s) { return ctrl0 + 8u * (MAX_STAGES + s); };
    auto tfull_bar = [&](int a) { return ctrl0 + 8u * (2 * MAX_STAGES + a); };
    auto tempty_bar = [&](int a) { return ctrl0 + 8u * (2 * MAX_STAGES + 2 + a); };
    const uint32_t epi_bar = ctrl0 + 8u * (2 * MAX_STAGES + 4);
    uint32_t *tmem_slot = (uint32_t *)(ctrl + 8 * (2 * MAX_STAGES + 5));
    volatile int *abort_flag = (volatile int *)(ctrl + 8 * (2 * MAX_STAGES + 5) + 4);

    // the shuffle tells the compiler that the warp number is the same in all lanes, so that the role code below
    // (loop counters, descriptors, TMA coordinates) can live in uniform registers
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(tfull_bar(a), 1);
            mbar_init(tempty_bar(a), 8);
        }
        mbar_init(epi_bar, 8);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == MMA_WARP) {
        tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    pdl_wait();                                            // set-up done: from here on the predecessor's results are read
    const uint32_t tmem_base = *tmem_slot;

    const int k_alloc = p.tiles_n * p.FT;     // row length of the float32 partial sums (split-K)
    const int total_tiles = p.tiles_m * p.tiles_n * p.splits;   // work items: (tile, K slice), slice fastest
    const int PQ = p.P * p.Q;

    if (warp < N_PRODUCERS) {
        // ------------------------------------------------------------------ producers
        // Issuing one TMA load costs the issuing thread about 300 cycles whatever the box size (measured), so
        // one warp cannot feed the tensor core.  Every producer warp walks the same sequence of pipeline
        // stages and fills those whose running index is congruent to its warp number.
        int stage = 0, turn = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < total_tiles && ok; item += gridDim.x) {
            // the divisions below are skipped in the common cases (no split-K, one filter tile) and done in
            // 32 bits when the pixel count allows: each costs this lone warp a few hundred cycles
            int tile = item, split = 0, it_begin = 0, it_end = p.iters;
            if (p.splits > 1) {
                tile = item / p.splits; split = item - tile * p.splits;
                it_begin = split * p.ipp; it_end = min(p.iters, it_begin + p.ipp);
            }
            int mt = tile, nt_f = 0;
            if (p.tiles_n > 1) { mt = tile / p.tiles_n; nt_f = tile - mt * p.tiles_n; }
            const long long m0 = (long long)mt * p.PT;
            int n_img, rem;
            if (p.M < (1ll << 31)) {
                n_img = (int)((uint32_t)m0 / (uint32_t)PQ);
                rem = (int)((uint32_t)m0 - (uint32_t)n_img * (uint32_t)PQ);
            } else {
                n_img = (int)(m0 / PQ);
                rem = (int)(m0 - (long long)n_img * PQ);
            }
            const int p0 = (int)((uint32_t)rem / (uint32_t)p.Q), q0 = rem - p0 * p.Q;
            const int wc = q0 * p.stride - p.pad, hc = p0 * p.stride - p.pad;
            if (p.small_c == 2) {
                // stride-2 stem read as pixel pairs: the tensor map sees [N][H][W/2][16]; a pair-tap is one im2col
                // load of PT pixels x 32 bytes = one K step; 4 pair-taps per stage
                const int taps = p.R * p.pair_taps;
                const int wcp = q0 - ((p.pad + 1) >> 1);
                for (int it = 0; it < p.iters - p.res_iters; ++it) {
                    const bool mine = turn == warp;
                    if (++turn == N_PRODUCERS) turn = 0;
                    if (mine) ok = __all_sync(0xffffffffu, mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status));
                    if (!ok) break;
                    if (mine && elect_one()) {
                        const uint32_t x_dst = base + (uint32_t)stage * stage_bytes;
                        int loads = taps - it * 4;
                        if (loads > 4) loads = 4;
                        mbar_expect_tx(full_bar(stage), (uint32_t)(loads * p.PT * 32 + p.FT * BK * 2));
                        for (int t = 0; t < loads; ++t) {
                            const int tap = it * 4 + t;
                            const int r = tap / p.pair_taps, tp = tap - r * p.pair_taps;
                            tma_load_im2col(x_dst + (uint32_t)(t * p.PT * 32), &tm_x, full_bar(stage), 0, wcp, hc, n_img,
                                            (uint16_t)tp, (uint16_t)r);
                        }
                        tma_load_3d(x_dst + x_bytes, &tm_w, full_bar(stage), it * BK, 0, nt_f * p.FT);
                    }
                    __syncwarp();
                    if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                }
            } else if (p.small_c) {
                // 8 taps x 8 channels per stage; every tap is its own im2col load of PT pixels x 16 bytes
                const int taps = p.R * p.S;
                for (int it = 0; it < p.iters - p.res_iters; ++it) {
                    const bool mine = turn == warp;
                    if (++turn == N_PRODUCERS) turn = 0;
                    if (mine) ok = __all_sync(0xffffffffu, mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status));
                    if (!ok) break;
                    if (mine && elect_one()) {
                        const uint32_t x_dst = base + (uint32_t)stage * stage_bytes;
                        int nt = taps - it * 8;
                        if (nt > 8) nt = 8;
                        const int loads = (nt + 1) & ~1;      // an odd last tap is loaded twice: the MMA reads 2 taps
                        mbar_expect_tx(full_bar(stage), (uint32_t)(loads * p.PT * 16 + p.FT * BK * 2));
                        for (int t = 0; t < loads; ++t) {
                            int tap = it * 8 + t;
                            if (tap >= taps) tap = taps - 1;  // finite filler; its weights are zero
                            const int r = tap / p.S, s = tap - r * p.S;
                            tma_load_im2col(x_dst + (uint32_t)(t * p.PT * 16), &tm_x, full_bar(stage), 0, wc, hc, n_img,
                                            (uint16_t)s, (uint16_t)r);
                        }
                        tma_load_3d(x_dst + x_bytes, &tm_w, full_bar(stage), it * BK, 0, nt_f * p.FT);
                    }
                    __syncwarp();
                    if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                }
            } else {
            // A single warp hides no latency, so this loop keeps (tap, channel block, r, s) as counters:
            // an integer division per K block would cost more than the loads it feeds.
            int tap = 0, cb = 0, r = 0, s = 0;
            if (it_begin) {
                tap = it_begin / p.cblks; cb = it_begin - tap * p.cblks;
                r = tap / p.S; s = tap - r * p.S;
            }
            const int it_last = it_end - (p.splits == 1 ? p.res_iters : 0);
            const int k0 = nt_f * p.FT;
            for (int it = it_begin; it < it_last; ++it) {
                const bool mine = turn == warp;
                if (++turn == N_PRODUCERS) turn = 0;
                if (mine) ok = __all_sync(0xffffffffu, mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status));
                if (!ok) break;
                if (mine && elect_one()) {
                    const uint32_t x_dst = base + (uint32_t)stage * stage_bytes;
                    const uint32_t fb = full_bar(stage);
                    mbar_expect_tx(fb, (uint32_t)stage_bytes);
                    tma_load_im2col(x_dst, &tm_x, fb, cb * BK, wc, hc, n_img, (uint16_t)s, (uint16_t)r);
                    tma_load_3d(x_dst + x_bytes, &tm_w, fb, cb * BK, tap, k0);
                }
                __syncwarp();
                if (++cb == p.cblks) {
                    cb = 0; ++tap;
                    if (++s == p.S) { s = 0; ++r; }
                }
                if (++stage == p.stages) { stage = 0; phase ^= 1u; }
            }
            }
            // residual blocks (ORIENT_FILT): the residual tile [PT pixels][64 filters] is the pixel-side
            // operand and a 64-column slice of the identity matrix the filter-side operand, so that the
            // MMA adds residual[pixel][k] to accumulator row k
            for (int j = 0; j < p.res_iters && ok; ++j) {
                const bool mine = turn == warp;
                if (++turn == N_PRODUCERS) turn = 0;
                if (mine) ok = __all_sync(0xffffffffu, mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status));
                if (!ok) break;
                if (mine && elect_one()) {
                    const uint32_t x_dst = base + (uint32_t)stage * stage_bytes;
                    mbar_expect_tx(full_bar(stage), (uint32_t)stage_bytes);
                    tma_load_2d(x_dst, &tm_res, full_bar(stage), j * BK, (int)m0);
                    tma_load_2d(x_dst + x_bytes, &tm_id, full_bar(stage), j * BK, 0);
                }
                __syncwarp();
                if (++stage == p.stages) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == MMA_WARP) {
        // ------------------------------------------------------------------ MMA issue
        // instruction descriptor: D float32, A and B bf16, both K-major, M = 128, N = filters or pixels
        const int mma_n = ORIENT == ORIENT_PIX ? p.FT : p.PT;
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(mma_n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        int stage = 0, acc = 0;
        uint32_t phase = 0, acc_phase = 0;
        bool ok = true;
        // This warp, too, runs alone on its scheduler: the loop below keeps the channel-block counter and the
        // operand descriptors of the current stage incrementally (no division, no descriptor rebuild per K block).
        const uint64_t dx0 = smem_desc_sw128(base), dw0 = smem_desc_sw128(base + (uint32_t)x_bytes);
        const uint64_t stage_step = (uint64_t)(stage_bytes >> 4);     // descriptor start addresses count 16-byte units
        uint64_t dx = dx0, dw = dw0;
        const int main_iters = p.iters - p.res_iters;
        const bool plain = p.small_c == 0;
        for (int item = blockIdx.x; item < total_tiles && ok; item += gridDim.x) {
            int it_begin = 0, it_end = p.iters;
            int cb = 0;
            if (p.splits > 1) {
                const int split = item % p.splits;
                it_begin = split * p.ipp;
                it_end = min(p.iters, it_begin + p.ipp);
                cb = it_begin % p.cblks;
            }
            ok = __all_sync(0xffffffffu, mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, p.status));
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(acc * ACC_STRIDE);
            uint32_t accumulate = 0;
            for (int it = it_begin; it < it_end; ++it) {
                ok = __all_sync(0xffffffffu, mbar_wait(full_bar(stage), phase, abort_flag, p.status));
                if (!ok) break;
                const bool res_it = it >= main_iters;
                if (plain || res_it) {
                    int nk = BK / 16;
                    if (res_it) {
                        int left = p.k_pad - (it - main_iters) * BK;
                        if (left > BK) left = BK;
                        nk = (left + 15) >> 4;
                    } else if (cb == p.cblks - 1) {
                        nk = p.ksteps_last;
                    }
                    if (elect_one()) {
#pragma unroll
                        for (int kk = 0; kk < BK / 16; ++kk) {
                            if (kk < nk) {
                                // 16 channels = 32 bytes further along the swizzled row: +2 in 16-byte units
                                if (ORIENT == ORIENT_PIX)
                                    umma_bf16(d_tmem, dx + (uint64_t)(2 * kk), dw + (uint64_t)(2 * kk), idesc, accumulate);
                                else
                                    umma_bf16(d_tmem, dw + (uint64_t)(2 * kk), dx + (uint64_t)(2 * kk), idesc, accumulate);
                                accumulate = 1;
                            }
                        }
                        umma_commit(empty_bar(stage));   // frees the stage once these MMAs have read it
                    }
                } else {
                    const uint32_t x_addr = base + (uint32_t)stage * stage_bytes;
                    int nk;
                    if (p.small_c == 2) {
                        nk = p.R * p.pair_taps - it * 4;
                        if (nk > 4) nk = 4;
                    } else {
                        int nt = p.R * p.S - it * 8;
                        if (nt > 8) nt = 8;
                        nk = (nt + 1) >> 1;
                    }
                    if (elect_one()) {
                        if (p.small_c == 2) {
                            // pixel operand: one pair-tap (16 channels) per MMA, pair-taps PT*32 bytes apart
                            for (int kk = 0; kk < nk; ++kk) {
                                const uint64_t dxp = smem_desc_sw32(x_addr + (uint32_t)kk * (uint32_t)p.PT * 32u);
                                if (ORIENT == ORIENT_PIX)
                                    umma_bf16(d_tmem, dxp, dw + (uint64_t)(2 * kk), idesc, accumulate);
                                else
                                    umma_bf16(d_tmem, dw + (uint64_t)(2 * kk), dxp, idesc, accumulate);
                                accumulate = 1;
                            }
                        } else {
                            // pixel operand: two taps (2 x 8 channels) per MMA, taps PT*16 bytes apart
                            const uint32_t tap_bytes = (uint32_t)p.PT * 16u;
                            for (int kk = 0; kk < nk; ++kk) {
                                const uint64_t dxi = smem_desc_interleaved(x_addr + (uint32_t)(2 * kk) * tap_bytes, tap_bytes);
                                if (ORIENT == ORIENT_PIX)
                                    umma_bf16(d_tmem, dxi, dw + (uint64_t)(2 * kk), idesc, accumulate);
                                else
                                    umma_bf16(d_tmem, dw + (uint64_t)(2 * kk), dxi, idesc, accumulate);
                                accumulate = 1;
                            }
                        }
                        umma_commit(empty_bar(stage));
                    }
                }
                accumulate = 1;
                __syncwarp();
                if (++cb == p.cblks) cb = 0;
                dx += stage_step; dw += stage_step;
                if (++stage == p.stages) { stage = 0; phase ^= 1u; dx = dx0; dw = dw0; }
            }
            if (ok && elect_one()) umma_commit(tfull_bar(acc));
            __syncwarp();
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        // Two warps share each quarter of the tensor-memory lanes (a warp may only read lanes 32*(warp%4)..+31):
        // `half` says which half of every group's columns this warp takes.
        const int quarter = warp & 3;
        const int half = (warp - FIRST_EPI_WARP) >> 2;
        const int trow = quarter * 32 + lane;          // accumulator row (pixel or filter) of this thread
        const bool store_thread = warp == FIRST_EPI_WARP && lane == 0;
        int acc = 0;
        uint32_t acc_phase = 0, epi_phase = 0;
        uint32_t group_counter = 0;                    // staged groups so far (selects the buffer)
        bool ok = true;
        // filter-major orientation: this thread's filter and its bias are the same for every tile
        const float filt_bias = (ORIENT == ORIENT_FILT && trow < p.k_pad) ? __ldg(p.bias + trow) : 0.f;
        // Bounded barrier among the eight epilogue warps (one arrival per warp).  Per staged group:
        // everyone writes buffer g%2, the store thread makes sure every earlier store has been read
        // out of shared memory, all meet here, then the store thread issues the stores of group g.
        // Buffer g%2 was last used by group g-2, whose store was confirmed read before barrier g-1.
        auto epi_sync = [&]() {
            __syncwarp();
            if (lane == 0) mbar_arrive(epi_bar);
            bool r = __all_sync(0xffffffffu, mbar_wait(epi_bar, epi_phase, abort_flag, p.status, false));
            epi_phase ^= 1u;
            return r;
        };
        for (int item = blockIdx.x; item < total_tiles && ok; item += gridDim.x) {
            int tile = item, split = 0;
            if (p.splits > 1) { tile = item / p.splits; split = item - tile * p.splits; }
            int mt = tile, nt = 0;
            if (p.tiles_n > 1) { mt = tile / p.tiles_n; nt = tile - mt * p.tiles_n; }
            const long long m0 = (long long)mt * p.PT;
            const int k_base = nt * p.FT;
            // the epilogue ignores the abort flag: all eight warps must take the same decisions,
            // and they all watch the same barriers
            ok = __all_sync(0xffffffffu, mbar_wait(tfull_bar(acc), acc_phase, abort_flag, p.status, false));
            if (!ok) break;
            tc_fence_after();
            const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * ACC_STRIDE);

            if (p.splits > 1) {
                // split-K: this CTA holds a partial sum; store it as float32, the finalize kernel adds
                // the slices in a fixed order and applies bias, residual and activation
                float *part = p.partial + (size_t)split * (size_t)p.M * k_alloc;
                if (ORIENT == ORIENT_PIX) {
                    const long long m = m0 + trow;
                    for (int c0 = half * 16; c0 < p.FT; c0 += 32) {
                        uint32_t v[16];
                        tmem_ld16(t_row + (uint32_t)c0, v);
                        tmem_ld_wait();
                        if (m < p.M) {
                            float4 *dst = (float4 *)(part + (size_t)m * k_alloc + k_base + c0);
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                dst[j] = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                                     __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
                        }
                    }
                } else {
                    const int k = trow;
                    if (quarter * 32 < p.k_pad) {
                        for (int c0 = half * 16; c0 < p.PT; c0 += 32) {
                            uint32_t v[16];
                            tmem_ld16(t_row + (uint32_t)c0, v);
                            tmem_ld_wait();
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                const long long m = m0 + c0 + j;
                                if (m < p.M) part[(size_t)m * k_alloc + k] = __uint_as_float(v[j]);
                            }
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(tempty_bar(acc));
            } else if (ORIENT == ORIENT_PIX) {
                // rows = pixels, columns = filters; groups of 64 filters
                const long long m = m0 + trow;
                const bool row_ok = m < p.M;
                const bool has_res = p.res != nullptr && row_ok;
                const int groups = (p.FT + 63) / 64;
                for (int g = 0; g < groups && ok; ++g) {
                    uint8_t *buf_ptr = smem + (staging0 - base) + (group_counter & 1u) * GROUP_BYTES;
                    const uint32_t buf = staging0 + (group_counter & 1u) * GROUP_BYTES;
                    const int cg = g * 64;                       // first filter column of the group
                    // this warp's half of the group: 32 filters = 64 contiguous bytes of the thread's row
                    const int ch = cg + half * 32;
                    bf16x8 rv[4];
                    if (has_res) {
                        const __nv_bfloat16 *rrow = p.res + (size_t)m * p.k_pad + k_base + ch;
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            if (k_base + ch + j * 8 < p.k_pad) rv[j] = ldg8((const bf16x8 *)(rrow + j * 8));
                    }
                    uint32_t v[32];
#pragma unroll
                    for (int sb = 0; sb < 2; ++sb)
                        if (ch + sb * 16 < p.FT) tmem_ld16(t_row + (uint32_t)(ch + sb * 16), v + sb * 16);
                    tmem_ld_wait();
                    if (g == groups - 1) {               // accumulator fully read: hand it back to the MMA warp
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(tempty_bar(acc));
                    }
#pragma unroll
                    for (int sb = 0; sb < 2; ++sb) {
                        const int c0 = ch + sb * 16;
                        if (c0 < p.FT) {
#pragma unroll
                            for (int h = 0; h < 2; ++h) {
                                float f[8];
                                const float4 b0 = __ldg((const float4 *)(p.bias + k_base + c0 + h * 8));
                                const float4 b1 = __ldg((const float4 *)(p.bias + k_base + c0 + h * 8 + 4));
                                const float bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
                                for (int j = 0; j < 8; ++j) f[j] = __uint_as_float(v[sb * 16 + h * 8 + j]) + bb[j];
                                if (has_res && k_base + c0 + h * 8 < p.k_pad) {
                                    float rf[8];
                                    unpack8(rv[sb * 2 + h], rf);
#pragma unroll
                                    for (int j = 0; j < 8; ++j) f[j] += rf[j];
                                }
#pragma unroll
                                for (int j = 0; j < 8; ++j) f[j] = apply_act(f[j], p.act);
                                const int chunk = half * 4 + sb * 2 + h;      // 16-byte chunk within the 128-byte staged row
                                if (POOL) {
                                    // the 2x2 window of a pixel lives in lanes l, l^1 (next column) and l^Q, l^Q^1
                                    // (next image row): Q is a power of two <= 16 here, so all four are in this warp
#pragma unroll
                                    for (int j = 0; j < 8; ++j) {
                                        f[j] = fmaxf(f[j], __shfl_xor_sync(0xffffffffu, f[j], 1));
                                        f[j] = fmaxf(f[j], __shfl_xor_sync(0xffffffffu, f[j], p.Q));
                                    }
                                    if ((lane & 1) == 0 && (lane & p.Q) == 0) {
                                        const int prow = (trow / (2 * p.Q)) * (p.Q >> 1) + ((trow & (p.Q - 1)) >> 1);
                                        *(bf16x8 *)(buf_ptr + sub_off(prow, chunk)) = pack8(f);
                                    }
                                } else {
                                    *(bf16x8 *)(buf_ptr + sub_off(trow, chunk)) = pack8(f);
                                }
                            }
                        }
                    }
                    fence_async_smem();
                    if (store_thread) tma_store_wait_read<0>();
                    ok = epi_sync();
                    if (!ok) break;
                    if (store_thread) {
                        if (k_base + cg < p.k_pad) tma_store_2d(&tm_y, buf, k_base + cg, (int)(POOL ? m0 >> 2 : m0));
                        tma_store_commit();
                    }
                    ++group_counter;
                }
            } else {
                // rows = filters, columns = pixels; groups of 64 pixels
                const int k = trow;                       // this thread's filter
                const bool k_ok = k < p.k_pad;
                const float bias = filt_bias;
                const int n_sub = (p.k_pad + SUB - 1) / SUB;       // sub-tiles that hold real filters
                const bool warp_has_work = quarter * 32 < p.k_pad; // all 32 filters of this warp may be padding
                const int groups = p.PT / 64;
                const int hk = (k >> 3) & 7;              // 16-byte chunk of this filter within its 128-byte row
                for (int g = 0; g < groups && ok; ++g) {
                    uint8_t *dst = smem + (staging0 - base) + (group_counter & 1u) * GROUP_BYTES + (k >> 6) * SUB_BYTES + (k & 7) * 2;
                    const uint32_t buf = staging0 + (group_counter & 1u) * GROUP_BYTES;
                    const long long mg = m0 + g * 64;
                    if (warp_has_work && POOL && p.Q == 32) {
                        // a row pair is the whole group: the first warp of the quarter pools all 64 pixels
                        if (half == 0) {
                            uint32_t v[64];
#pragma unroll
                            for (int c = 0; c < 4; ++c) tmem_ld16(t_row + (uint32_t)(g * 64 + c * 16), v + c * 16);
                            tmem_ld_wait();
                            if (k_ok) {
                                float f[64];
#pragma unroll
                                for (int j = 0; j < 64; ++j) f[j] = apply_act(__uint_as_float(v[j]) + bias, p.act);
                                uint8_t *pd = smem + (staging0 - base) + (group_counter & 1u) * GROUP_BYTES + (k >> 6) * POOL_SUB_BYTES + (k & 7) * 2;
                                store_pooled<32, 64>(f, pd, hk, 0);
                            }
                        }
                    } else if (warp_has_work && POOL) {
                        // this warp's 32 pixels of the group (whole row pairs) for this filter, then their 8 pooled values
                        uint32_t v[32];
#pragma unroll
                        for (int c = 0; c < 2; ++c) tmem_ld16(t_row + (uint32_t)(g * 64 + half * 32 + c * 16), v + c * 16);
                        tmem_ld_wait();
                        if (k_ok) {
                            float f[32];
#pragma unroll
                            for (int j = 0; j < 32; ++j) f[j] = apply_act(__uint_as_float(v[j]) + bias, p.act);
                            uint8_t *pd = smem + (staging0 - base) + (group_counter & 1u) * GROUP_BYTES + (k >> 6) * POOL_SUB_BYTES + (k & 7) * 2;
                            switch (p.Q) {
                                case 2: store_pooled<2, 32>(f, pd, hk, half * 8); break;
                                case 4: store_pooled<4, 32>(f, pd, hk, half * 8); break;
                                case 8: store_pooled<8, 32>(f, pd, hk, half * 8); break;
                                default: store_pooled<16, 32>(f, pd, hk, half * 8); break;
                            }
                        }
                    } else if (warp_has_work) {
                        uint32_t v[32];
#pragma unroll
                        for (int c = 0; c < 2; ++c) tmem_ld16(t_row + (uint32_t)(g * 64 + half * 32 + c * 16), v + c * 16);
                        tmem_ld_wait();
                        if (k_ok) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                float f = __uint_as_float(v[j]) + bias;
                                f = apply_act(f, p.act);
                                *(__nv_bfloat16 *)(dst + sub_off(half * 32 + j, hk)) = __float2bfloat16_rn(f);
                            }
                        }
                    }
                    if (g == groups - 1) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(tempty_bar(acc));
                    }
                    fence_async_smem();
                    if (store_thread) tma_store_wait_read<0>();
                    ok = epi_sync();
                    if (!ok) break;
                    if (store_thread) {
                        for (int sb = 0; sb < n_sub; ++sb) {
                            if (POOL) tma_store_2d(&tm_y, buf + sb * POOL_SUB_BYTES, sb * SUB, (int)(mg >> 2));
                            else tma_store_2d(&tm_y, buf + sb * SUB_BYTES, sb * SUB, (int)mg);
                        }
                        tma_store_commit();
                    }
                    ++group_counter;
                }
            }
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (store_thread) tma_store_wait_all();          // staged data must be read before the CTA's memory goes away
    }

    // ---------------------------------------------------------------------- teardown
    if (*abort_flag) {
        // give copies that may still be in flight time to land before the CTA's memory is released
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == MMA_WARP) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------------ host

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
typedef CUresult (*EncodeIm2colFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const int *, const int *, cuuint32_t, cuuint32_t,
                                   const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn g_encode_tiled = nullptr;
static EncodeIm2colFn g_encode_im2col = nullptr;
static int g_driver_version = 0;

static cprune_status load_driver_entry_points() {
    static std::mutex mu;
    std::lock_guard<std::mutex> lock(mu);
    if (g_encode_tiled && g_encode_im2col) return CPRUNE_OK;
    cudaDriverEntryPointQueryResult q;
    void *fn = nullptr;
    CPRUNE_CUDA_CHECK(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
    if (!fn || q != cudaDriverEntryPointSuccess) return cuda_fail(cudaErrorUnknown, "cuTensorMapEncodeTiled not found");
    g_encode_tiled = (EncodeTiledFn)fn;
    fn = nullptr;
    CPRUNE_CUDA_CHECK(cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &fn, cudaEnableDefault, &q));
    if (!fn || q != cudaDriverEntryPointSuccess) return cuda_fail(cudaErrorUnknown, "cuTensorMapEncodeIm2col not found");
    g_encode_im2col = (EncodeIm2colFn)fn;
    CPRUNE_CUDA_CHECK(cudaDriverGetVersion(&g_driver_version));
    return CPRUNE_OK;
}

// Split-K finalize: y[m][k] = act(bias[k] + residual[m][k] + sum over slices of partial[s][m][k]),
// slices added in a fixed order (deterministic).  Four threads per (conv pixel, 8 filters).  With
// pool_q > 0 an output pixel is the maximum over its 2x2 window of conv pixels (image rows of pool_q
// pixels; a pooled pixel j of an image covers conv pixels 2*(j / (pool_q/2))*pool_q + 2*(j % (pool_q/2)) + {0,1,pool_q,pool_q+1}).
__global__ void __launch_bounds__(256) splitk_finalize_kernel(const float *__restrict__ partial, int splits, long long M,
                                                              int k_alloc, int k8, const float *__restrict__ bias,
                                                              const bf16x8 *__restrict__ res, int act, int pool_q,
                                                              bf16x8 *__restrict__ y) {
    pdl_trigger();
    pdl_wait();
    // Four lanes share one (conv pixel, 8 filters): lane L adds slices L, L + 4, ... in index order and the four sums are
    // combined as (L0 + L1) + (L2 + L3): a fixed order, so the result does not depend on timing.  With a pool the four
    // conv pixels of a window sit in four such lane groups (16 lanes per output).
    const int windows = pool_q ? 4 : 1;
    const int lanes_per_out = 4 * windows;
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long e = t / lanes_per_out;                      // output element group (pixel, 8 filters)
    const int sub = (int)(t - e * lanes_per_out);
    const int L = sub & 3, wdx = sub >> 2;
    const long long out_pixels = pool_q ? M / 4 : M;
    const bool valid = e < out_pixels * k8;                     // whole lane groups are valid or not (uniform shuffles below)
    const long long ec = valid ? e : 0;
    const long long mo = ec / k8;
    const int kg = (int)(ec - mo * k8);
    const int hq = pool_q >> 1;
    long long m = mo;
    if (pool_q) m = 2 * (mo / hq) * pool_q + 2 * (mo % hq) + (wdx & 1) + (wdx >> 1) * pool_q;
    float f[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) f[j] = 0.f;
    for (int sidx = L; sidx < splits; sidx += 4) {
        const float4 *src = (const float4 *)(partial + ((size_t)sidx * M + m) * k_alloc + kg * 8);
        const float4 a = __ldg(src), b = __ldg(src + 1);
        f[0] += a.x; f[1] += a.y; f[2] += a.z; f[3] += a.w;
        f[4] += b.x; f[5] += b.y; f[6] += b.z; f[7] += b.w;
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        f[j] += __shfl_xor_sync(0xffffffffu, f[j], 1);
        f[j] += __shfl_xor_sync(0xffffffffu, f[j], 2);
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) f[j] += __ldg(bias + kg * 8 + j);
    if (res) {
        float rf[8];
        unpack8(ldg8(res + m * k8 + kg), rf);
#pragma unroll
        for (int j = 0; j < 8; ++j) f[j] += rf[j];
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) f[j] = apply_act(f[j], act);
    if (pool_q) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            f[j] = fmaxf(f[j], __shfl_xor_sync(0xffffffffu, f[j], 4));
            f[j] = fmaxf(f[j], __shfl_xor_sync(0xffffffffu, f[j], 8));
        }
    }
    if (valid && sub == 0) y[e] = pack8(f);
}

// 128 x 128 identity in bf16 (1.0 = 0x3F80): the filter-side operand of the residual blocks (see the producer).
// Initialised in the library image, so no launch and no synchronisation is needed before its first use.
struct IdentityBits {
    uint16_t v[128 * 128];
    constexpr IdentityBits() : v{} {
        for (int i = 0; i < 128; ++i) v[i * 128 + i] = 0x3F80;
    }
};
static __device__ __align__(256) const IdentityBits g_identity = IdentityBits();

// Device address of the identity matrix on the current device (looked up once per device).
static cprune_status identity_address(void **out) {
    static std::mutex mu;
    static void *ptrs[64] = {nullptr};
    int dev = 0;
    CPRUNE_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return CPRUNE_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(mu);
    if (!ptrs[dev]) {
        void *p = nullptr;
        CPRUNE_CUDA_CHECK(cudaGetSymbolAddress(&p, g_identity));
        ptrs[dev] = p;
    }
    *out = ptrs[dev];
    return CPRUNE_OK;
}

// Tiled bf16 tensor map without swizzle (used by the depthwise kernel for its input patches).
cprune_status encode_tiled_bf16(CUtensorMap *map, const void *ptr, int rank, const unsigned long long *dims,
                                const unsigned long long *strides_bytes, const unsigned *box) {
    cprune_status st = load_driver_entry_points();
    if (st != CPRUNE_OK) return st;
    cuuint64_t d[5], s[4];
    cuuint32_t b[5], e[5];
    for (int i = 0; i < rank; ++i) { d[i] = dims[i]; b[i] = box[i]; e[i] = 1; }
    for (int i = 0; i + 1 < rank; ++i) s[i] = strides_bytes[i];
    CUresult r = g_encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void *>(ptr), d, s, b, e,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled(depthwise)");
    return CPRUNE_OK;
}

cprune_status encode_tiled_bf16_swz(CUtensorMap *map, const void *ptr, int rank, const unsigned long long *dims,
                                    const unsigned long long *strides_bytes, const unsigned *box, int swizzle_bytes, bool for_loads) {
    cprune_status st = load_driver_entry_points();
    if (st != CPRUNE_OK) return st;
    cuuint64_t d[5], s[4];
    cuuint32_t b[5], e[5];
    for (int i = 0; i < rank; ++i) { d[i] = dims[i]; b[i] = box[i]; e[i] = 1; }
    for (int i = 0; i + 1 < rank; ++i) s[i] = strides_bytes[i];
    CUresult r = g_encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void *>(ptr), d, s, b, e,
                                CU_TENSOR_MAP_INTERLEAVE_NONE,
                                swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : (swizzle_bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE),
                                for_loads ? CU_TENSOR_MAP_L2_PROMOTION_L2_128B : CU_TENSOR_MAP_L2_PROMOTION_NONE,
                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    return CPRUNE_OK;
}

static int smem_for(int stages, int PT, int FT, int staging_bufs, int group_rows) {
    (void)group_rows;
    return 1024 /* alignment slack */ + stages * (PT + FT) * BK * 2 + staging_bufs * GROUP_BYTES + CTRL_BYTES;
}

// Chooses orientation, tiles and pipeline depth.  Eligible: dense, im2col corner limits.
cprune_status plan_conv_tensor(cprune_plan *plan) {
    cprune_plan_info &i = plan->info;
    if (i.groups != 1) return CPRUNE_ERR_UNSUPPORTED;
    // stride-1 tasks with more than one tap: patch kernel when its tile is well filled
    plan->patch = 0;
    if (!(plan->opts.flags & CPRUNE_FLAG_IM2COL_ONLY) && plan_conv_patch(plan) == CPRUNE_OK) return CPRUNE_OK;
    if (i.R > 16 || i.S > 16 || i.pad > 64 || i.stride > 8) return CPRUNE_ERR_UNSUPPORTED;
    if (i.W > 65535 || i.H > 65535) return CPRUNE_ERR_UNSUPPORTED;
    const long long M = (long long)i.N * i.P * i.Q;
    const int k16 = round_up(i.K, 16);
    int PT, FT, tiles_n, bufs, group_rows;
    plan->small_c = (i.c_pad == 8 && i.K <= 128 && i.R * i.S > 1) ? 1 : 0;
    // stride-2 stems with odd pad and odd S: read the image as pixel pairs (16 channels per pair), which halves
    // the number of loads and doubles their row width; the packed filters get one zero tap in front of each row
    if (plan->small_c && i.stride == 2 && (i.W & 1) == 0 && (i.pad & 1) == 1 && (i.S & 1) == 1) plan->small_c = 2;
    plan->s_packed = plan->small_c == 2 ? i.S + 1 : i.S;
    // Orientation.  K <= 128: filters on the 128-row side (256 pixels per MMA) -- except for tasks with one or two
    // K blocks and at most 32 filters (MobileNetV2 project layers), where the pixel-major epilogue, in which every
    // thread stores one pixel's contiguous filters, is faster than the transposing one (measured: 45 vs 62 us).
    const int k_blocks = i.R * i.S * ((i.c_pad + BK - 1) / BK);
    const bool few_filters = !plan->small_c && k_blocks <= 2 && i.K <= 32;
    if (i.K <= 128 && !few_filters) {
        // filters on the MMA-M side (padded to 128 rows), 256 pixels on the MMA-N side
        plan->orient = ORIENT_FILT;
        PT = 256; FT = 128; tiles_n = 1; bufs = 2; group_rows = 64;
    } else {
        plan->orient = ORIENT_PIX;
        PT = 128; group_rows = 128; bufs = 2;
        const int tiles_m = (int)ceil_div(M, PT);
        // fewest filter tiles that fit the 256-column accumulator, then split further while that
        // fills more of the 148 SMs without dropping below 128 filters per tile
        tiles_n = (k16 + 255) / 256;
        while (true) {
            int next = tiles_n + 1;
            int ft_next = round_up((k16 + next - 1) / next, 64);
            if (ft_next < 128) break;
            if ((long long)tiles_m * tiles_n >= 148) break;
            tiles_n = next;
        }
        // with several filter tiles every tile must end on a 64-filter boundary: the staged stores
        // are 64 filters wide and only the tensor's own edge clips them
        FT = round_up((k16 + tiles_n - 1) / tiles_n, tiles_n > 1 ? 64 : 16);
        tiles_n = (k16 + FT - 1) / FT;
    }
    int stages = MAX_STAGES;
    while (stages > 2 && smem_for(stages, PT, FT, bufs, group_rows) > 227 * 1024) --stages;
    i.tile_m = PT;
    i.tile_n = FT;
    i.tile_k = BK;
    i.stages = stages;
    i.tiles_m = (int)ceil_div(M, PT);
    i.tiles_n = tiles_n;
    i.k_alloc = tiles_n * FT;
    const int cblks = (i.c_pad + BK - 1) / BK;
    const int ksteps = (cblks - 1) * (BK / 16) + (i.c_pad - (cblks - 1) * BK + 15) / 16;
    i.padded_flops = 2.0 * (double)i.tiles_m * PT * (double)i.k_alloc * (double)(i.R * i.S) * ksteps * 16.0;
    if (plan->small_c == 1) i.padded_flops = 2.0 * (double)i.tiles_m * PT * (double)i.k_alloc * ((i.R * i.S + 1) / 2) * 16.0;
    if (plan->small_c == 2) i.padded_flops = 2.0 * (double)i.tiles_m * PT * (double)i.k_alloc * (i.R * (i.S + 1) / 2) * 16.0;
    plan->staging_bufs = bufs;
    plan->smem_bytes = smem_for(stages, PT, FT, bufs, group_rows);
    // Split-K when the tiles cannot fill the SMs: slices of the K blocks go to different CTAs, which
    // store float32 partial sums; a small second kernel adds them.  The choice minimises a cost model
    // fitted to measurements on B200 (microseconds): waves x (K blocks per slice x time per block +
    // per-item overhead) + launch floor (+ the second pass).
    plan->splits = 1;
    const int iters = i.R * i.S * cblks;
    const long long tiles = (long long)i.tiles_m * tiles_n;
    if (!plan->small_c && tiles <= 100 && iters >= 4) {
        const double blk = plan->orient == ORIENT_PIX ? (FT > 128 ? 0.375 * FT / 128.0 : 0.375) : 0.45;
        auto cost = [&](int sp) {
            const int ipp = (iters + sp - 1) / sp;
            return (double)ceil_div(tiles * sp, 148) * (ipp * blk + 4.0) + 6.0 + (sp > 1 ? 2.5 : 0.0);
        };
        double best = cost(1);
        for (int sp = 2; sp <= 16 && sp * 2 <= iters; ++sp) {
            const int ipp = (iters + sp - 1) / sp;
            if ((sp - 1) * ipp >= iters) continue;              // a slice would be empty
            if ((double)sp * M * i.k_alloc * 4.0 > 256e6) break; // keep the partial sums within L2 reach
            const double t = cost(sp);
            if (t < best * 0.9) { best = t; plan->splits = sp; }
        }
    }
    // A 2x2 max-pool is fused when a tile holds whole pairs of image rows: Q a power of two with the
    // four pixels of a window in one warp (pixel-major: Q <= 16) or in one thread's 64-pixel group
    // (filter-major: Q <= 32).  The split-K finalize kernel pools for any even P, Q.
    plan->fused_pool = 0;
    if (plan->opts.pool == CPRUNE_POOL_MAX2X2) {
        const bool pow2 = (i.Q & (i.Q - 1)) == 0 && i.Q >= 2;
        if (plan->splits > 1) plan->fused_pool = 1;
        else if (pow2 && i.Q <= (plan->orient == ORIENT_PIX ? 16 : 32)) plan->fused_pool = 1;
    }
    plan->ipp = (iters + plan->splits - 1) / plan->splits;
    plan->partial_bytes = plan->splits > 1 ? (size_t)plan->splits * (size_t)M * i.k_alloc * 4 : 0;
    {
        // estimate: per K block the tensor pipe needs 4 MMAs of N / 2 cycles, shared memory takes the TMA writes of
        // both operands and the MMAs' operand reads at 128 bytes per clock; about 1.9 GHz; launch and drain on top
        const int mma_n = plan->orient == ORIENT_PIX ? FT : PT;
        const double tensor = 4.0 * mma_n / 2.0;
        const double smem = (PT + FT) * 128.0 / 128.0 + 4.0 * (128.0 + mma_n) * 32.0 / 128.0;
        const double per_block = tensor > smem ? tensor : smem;
        const double waves = (double)ceil_div(tiles * plan->splits, 148);
        plan->est_us = waves * (plan->ipp * per_block + 2000.0) / 1900.0 + 4.0 + (plan->splits > 1 ? 3.0 : 0.0);
    }
    return CPRUNE_OK;
}

static cprune_status encode_maps(cprune_plan *plan, const void *x, const void *w, void *y, const void *res) {
    const cprune_plan_info &i = plan->info;
    cprune_status st = load_driver_entry_points();
    if (st != CPRUNE_OK) return st;
    if (plan->map_x != x) {
        cuuint64_t dims[4] = {(cuuint64_t)i.c_pad, (cuuint64_t)i.W, (cuuint64_t)i.H, (cuuint64_t)i.N};
        cuuint64_t strides[3] = {(cuuint64_t)i.c_pad * 2, (cuuint64_t)i.W * i.c_pad * 2, (cuuint64_t)i.H * i.W * i.c_pad * 2};
        int lower[2] = {-i.pad, -i.pad};
        int upper[2] = {i.pad - (i.S - 1), i.pad - (i.R - 1)};
        cuuint32_t estr[4] = {1, (cuuint32_t)i.stride, (cuuint32_t)i.stride, 1};
        cuuint32_t chans = BK;
        CUtensorMapSwizzle swz = CU_TENSOR_MAP_SWIZZLE_128B;
        if (plan->small_c == 1) {          // 8 channels (16 bytes) per pixel, dense rows, no swizzle
            chans = 8;
            swz = CU_TENSOR_MAP_SWIZZLE_NONE;
        } else if (plan->small_c == 2) {   // the same memory seen as [N][H][W/2][16]: pixel pairs, unit step along W/2
            dims[0] = 16; dims[1] = (cuuint64_t)i.W / 2;
            strides[0] = 32;
            lower[0] = -((i.pad + 1) / 2);
            upper[0] = i.Q - i.W / 2 + lower[0];   // exactly Q start positions per image row
            estr[1] = 1;
            chans = 16;
            swz = CU_TENSOR_MAP_SWIZZLE_32B;
        }
        CUresult r = g_encode_im2col(&plan->tm_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(x), dims, strides,
                                     lower, upper, chans, (cuuint32_t)i.tile_m, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                                     CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeIm2col");
        // Drivers up to 13.1 set a descriptor bit for im2col maps of tensors smaller than 128 KiB
        // that makes the load misbehave; the open-source CUTLASS im2col path clears it the same way.
        const size_t bytes = (size_t)i.N * i.H * i.W * i.c_pad * 2;
        if (g_driver_version <= 13010 && bytes < 131072) reinterpret_cast<uint64_t *>(&plan->tm_a)[1] &= ~(1ull << 21);
        plan->map_x = x;
    }
    if (plan->map_w != w) {
        // small-C modes read a filter row [R * s_packed taps][8 channels] as one long channel axis
        const int row_elems = i.R * plan->s_packed * i.c_pad;
        cuuint64_t dims[3] = {(cuuint64_t)(plan->small_c ? row_elems : i.c_pad), (cuuint64_t)(plan->small_c ? 1 : i.R * i.S),
                              (cuuint64_t)i.k_alloc};
        cuuint64_t strides[2] = {(cuuint64_t)(plan->small_c ? row_elems : i.c_pad) * 2, (cuuint64_t)row_elems * 2};
        cuuint32_t box[3] = {BK, 1, (cuuint32_t)i.tile_n};
        cuuint32_t estr[3] = {1, 1, 1};
        CUresult r = g_encode_tiled(&plan->tm_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(w), dims, strides, box,
                                    estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                    CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled(w)");
        plan->map_w = w;
    }
    if (plan->map_y != y) {
        // output as a 2-D tensor [pixels][k_pad]; stored in boxes of 64 filters x 128 or 64 pixels
        // (with a fused 2x2 pool: [pooled pixels][k_pad], boxes of 32 or 16 pooled pixels)
        const long long M = (long long)i.N * i.P * i.Q / (plan->fused_pool ? 4 : 1);
        cuuint64_t dims[2] = {(cuuint64_t)i.k_pad, (cuuint64_t)M};
        cuuint64_t strides[1] = {(cuuint64_t)i.k_pad * 2};
        cuuint32_t box[2] = {SUB, (cuuint32_t)((plan->orient == ORIENT_PIX ? 128 : 64) / (plan->fused_pool ? 4 : 1))};
        cuuint32_t estr[2] = {1, 1};
        CUresult r = g_encode_tiled(&plan->tm_y, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, y, dims, strides, box, estr,
                                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                    CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled(y)");
        plan->map_y = y;
    }
    if (plan->orient == ORIENT_FILT && res && plan->map_res != res) {
        // residual [pixels][k_pad], loaded as the pixel-side operand: 64 filters x 256 pixels
        const long long M = (long long)i.N * i.P * i.Q;
        cuuint64_t dims[2] = {(cuuint64_t)i.k_pad, (cuuint64_t)M};
        cuuint64_t strides[1] = {(cuuint64_t)i.k_pad * 2};
        cuuint32_t box[2] = {BK, (cuuint32_t)i.tile_m};
        cuuint32_t estr[2] = {1, 1};
        CUresult r = g_encode_tiled(&plan->tm_res, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(res), dims, strides,
                                    box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                    CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled(res)");
        void *ident = nullptr;
        cprune_status s2 = identity_address(&ident);
        if (s2 != CPRUNE_OK) return s2;
        cuuint64_t idims[2] = {128, 128};
        cuuint64_t istrides[1] = {256};
        cuuint32_t ibox[2] = {BK, 128};
        r = g_encode_tiled(&plan->tm_id, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, ident, idims, istrides, ibox, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled(identity)");
        plan->map_res = res;
    }
    return CPRUNE_OK;
}

cprune_status launch_splitk_finalize(const float *partial, int splits, long long M, int k_alloc, int k_pad, const float *bias,
                                     const void *res, int act, void *y, cudaStream_t st) {
    const long long threads = M * (k_pad / 8) * 4;
    CPRUNE_CUDA_CHECK(launch_chained(splitk_finalize_kernel, dim3((unsigned)ceil_div(threads, 256)), dim3(256), 0, st, partial, splits, M,
                                     k_alloc, k_pad / 8, bias, (const bf16x8 *)res, act, 0, (bf16x8 *)y));
    return CPRUNE_OK;
}

static int sm_count() {
    static int n = 0;
    if (!n) {
        int dev = 0;
        cudaGetDevice(&dev);
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    }
    return n;
}

cprune_status launch_conv_tensor(cprune_plan *plan, const void *x, const void *w, const float *b, const void *res,
                                 void *y, void *partial, cudaStream_t st, bool input_regrouped) {
    const cprune_plan_info &i = plan->info;
    if (plan->patch) return launch_conv_patch(plan, x, w, b, res, y, partial, st, input_regrouped);
    CUtensorMap tm_x, tm_w, tm_y, tm_res, tm_id;
    const bool split = plan->splits > 1;
    if (split && !partial) return CPRUNE_ERR_INVALID_ARG;
    const bool mma_res = plan->orient == ORIENT_FILT && res != nullptr && !split;
    {
        std::lock_guard<std::mutex> lock(plan->mu);
        if (plan->map_x != x || plan->map_w != w || plan->map_y != y || (mma_res && plan->map_res != res)) {
            cprune_status s = encode_maps(plan, x, w, y, res);
            if (s != CPRUNE_OK) return s;
        }
        std::memcpy(&tm_x, &plan->tm_a, sizeof(CUtensorMap));
        std::memcpy(&tm_w, &plan->tm_b, sizeof(CUtensorMap));
        std::memcpy(&tm_y, &plan->tm_y, sizeof(CUtensorMap));
        // without a tensor-core residual the two extra maps are never read; pass valid copies anyway
        std::memcpy(&tm_res, mma_res ? &plan->tm_res : &plan->tm_y, sizeof(CUtensorMap));
        std::memcpy(&tm_id, mma_res ? &plan->tm_id : &plan->tm_y, sizeof(CUtensorMap));
    }
    static std::mutex attr_mu;
    static int attr_set[64] = {0};     // the shared-memory limit of a kernel is a per-device attribute
    {
        int dev = 0;
        CPRUNE_CUDA_CHECK(cudaGetDevice(&dev));
        if (dev < 0 || dev >= 64) return CPRUNE_ERR_UNSUPPORTED;
        std::lock_guard<std::mutex> lock(attr_mu);
        if (!attr_set[dev]) {
            CPRUNE_CUDA_CHECK(cudaFuncSetAttribute(conv_tc_kernel<ORIENT_PIX, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            CPRUNE_CUDA_CHECK(cudaFuncSetAttribute(conv_tc_kernel<ORIENT_PIX, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            CPRUNE_CUDA_CHECK(cudaFuncSetAttribute(conv_tc_kernel<ORIENT_FILT, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            CPRUNE_CUDA_CHECK(cudaFuncSetAttribute(conv_tc_kernel<ORIENT_FILT, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            attr_set[dev] = 1;
        }
    }
    TcParams p;
    p.M = (long long)i.N * i.P * i.Q;
    p.P = i.P; p.Q = i.Q; p.stride = i.stride; p.pad = i.pad; p.R = i.R; p.S = i.S;
    p.cblks = (i.c_pad + BK - 1) / BK;
    p.ksteps_last = (i.c_pad - (p.cblks - 1) * BK + 15) / 16;
    p.PT = i.tile_m; p.FT = i.tile_n; p.tiles_m = i.tiles_m; p.tiles_n = i.tiles_n; p.k_pad = i.k_pad; p.stages = i.stages;
    p.small_c = plan->small_c;
    p.pair_taps = (i.S + 1) / 2;
    p.splits = plan->splits;
    p.pool = plan->fused_pool;
    p.ipp = plan->ipp;
    p.partial = (float *)partial;
    p.res_iters = mma_res ? (i.k_pad + BK - 1) / BK : 0;
    const int main_iters = plan->small_c == 2 ? (i.R * p.pair_taps + 3) / 4
                           : plan->small_c == 1 ? (i.R * i.S + 7) / 8 : i.R * i.S * p.cblks;
    p.iters = main_iters + p.res_iters;
    if (plan->splits == 1) p.ipp = p.iters;   // one slice covers everything, the residual blocks included
    p.act = plan->opts.activation;
    p.bias = b;
    p.res = (mma_res || split) ? nullptr : (const __nv_bfloat16 *)res;   // ORIENT_PIX adds it in the epilogue
    p.status = device_status_word();
    if (!p.status) return cuda_fail(cudaGetLastError(), "status word");
    const int total = i.tiles_m * i.tiles_n * plan->splits;
    if (total == 0) return CPRUNE_OK;
    const int grid = total < sm_count() ? total : sm_count();
    const bool pool_in_kernel = plan->fused_pool && !split;
    if (plan->orient == ORIENT_PIX) {
        if (pool_in_kernel) CPRUNE_CUDA_CHECK(launch_chained(conv_tc_kernel<ORIENT_PIX, 1>, dim3(grid), dim3(TC_THREADS), (size_t)plan->smem_bytes, st, tm_x, tm_w, tm_y, tm_res, tm_id, p));
        else CPRUNE_CUDA_CHECK(launch_chained(conv_tc_kernel<ORIENT_PIX, 0>, dim3(grid), dim3(TC_THREADS), (size_t)plan->smem_bytes, st, tm_x, tm_w, tm_y, tm_res, tm_id, p));
    } else {
        if (pool_in_kernel) CPRUNE_CUDA_CHECK(launch_chained(conv_tc_kernel<ORIENT_FILT, 1>, dim3(grid), dim3(TC_THREADS), (size_t)plan->smem_bytes, st, tm_x, tm_w, tm_y, tm_res, tm_id, p));
        else CPRUNE_CUDA_CHECK(launch_chained(conv_tc_kernel<ORIENT_FILT, 0>, dim3(grid), dim3(TC_THREADS), (size_t)plan->smem_bytes, st, tm_x, tm_w, tm_y, tm_res, tm_id, p));
    }
    CPRUNE_LAUNCH_CHECK("conv_tc_kernel");
    if (split) {
        const long long elems = (plan->fused_pool ? p.M / 4 : p.M) * (i.k_pad / 8) * (plan->fused_pool ? 16 : 4);   // threads
        CPRUNE_CUDA_CHECK(launch_chained(splitk_finalize_kernel, dim3((unsigned)ceil_div(elems, 256)), dim3(256), 0, st, (const float *)partial,
                                         plan->splits, p.M, i.k_alloc, i.k_pad / 8, b, (const bf16x8 *)res, plan->opts.activation,
                                         plan->fused_pool ? i.Q : 0, (bf16x8 *)y));
    }
    return CPRUNE_OK;
}

}  // namespace cprune
