// Fused inverted-residual block (MobileNetV2 / MnasNet, paper Sec. 4.1): 1x1 expand + activation, 3x3 depthwise
// (stride 1, pad 1) + activation, 1x1 project (+ the block's input as residual), as ONE kernel.  The expanded
// ("hidden") tensor, which is six times wider than the block's input and which the three separate tasks write
// and read four times, never leaves the SM: it lives in tensor memory and shared memory, 64 channels at a time.
//
// One CTA per image (H * W <= 256 pixels, i.e. the 14x14 and 7x7 stages) and per slice of the hidden channels,
// 16 warps, no role split: the phases of a 64-channel chunk of the hidden tensor follow each other, and only the
// project MMAs of a chunk overlap the expand phase of the next.  A block is a chain of short dependent phases, so
// its time is latency, not throughput: with `splits` > 1 the chunks of an image are dealt to that many CTAs, each
// of which leaves a float32 partial sum of the project layer in the workspace, and the split-reduction finalize
// kernel of the tensor family adds the slices in a fixed order and applies bias, residual and activation.
//   X   [pixels][C_in]  the image, loaded once by TMA as the row operand of the expand MMAs (128-byte swizzled
//       rows, one 64-channel block after the other); it is also the residual of the last phase;
//   per chunk h:
//     expand   acc1[pixel][64]  = X x We[h]^T                       tcgen05.mma, accumulator in tensor memory
//     stage 1  H1 = act(acc1 + be) as bf16 into a (H+2) x (W+2) x 64 image with a zero border in shared memory
//     depthwise H2[pixel][64]   = act(sum of 9 taps of H1 x Wd + bd) on the CUDA cores, float32, written as bf16
//              in the row-operand layout of an MMA
//     project  acc2[pixel][C_out] += H2 x Wp[:, h]^T                 tcgen05.mma
//   last: y = act_out(acc2 + bp + X) as bf16, staged in shared memory and copied out in whole 16-byte pieces (an
//   image's output is one contiguous range of y).
// bf16 roundings happen where the three separate tasks would store bf16, so the result equals theirs up to the order
// of float32 additions.  Every wait is bounded (see sm100_ptx.cuh).
#include <cuda.h>

#include <array>
#include <cstring>
#include <map>
#include <mutex>

#include "common.cuh"
#include "plan.h"
#include "sm100_ptx.cuh"

struct cprune_block {
    cprune_block_info info;
    int refs = 0;
    int MB = 0, cblks = 0, nk_last = 0, nchunks = 0, smem_bytes = 0, splits = 1;
    std::mutex mu;
    const void *map_x = nullptr, *map_w = nullptr;
    alignas(64) CUtensorMap tm_x, tm_we, tm_wp;
};

namespace cprune {

constexpr int FB_THREADS = 512;
constexpr int FB_CHUNK = 64;               // hidden channels per chunk = one 128-byte operand row

struct BlockParams {
    int HW, H, W, MB, cblks, nk_last, nchunks, hid_alloc, k_alloc, k_pad, act, act_out, residual;
    int splits;                            // CTAs per image; CTA r of an image takes chunks r, r + splits, ...
    float *partial;                        // splits > 1: float32 partial sums [splits][N * HW][k_alloc]
    long long M;                           // N * HW
    const float *be, *bd, *bp;             // float32 biases: expand [hid_alloc], depthwise [hid_alloc], project [k_alloc]
    const bf16x8 *wd;                      // depthwise taps [9][hid_alloc / 8]
    bf16x8 *y;
    int *status;
};

__device__ __forceinline__ float act_apply(float v, int act) {
    if (act == CPRUNE_ACT_RELU) return fmaxf(v, 0.f);
    if (act == CPRUNE_ACT_RELU6) return fminf(fmaxf(v, 0.f), 6.f);
    return v;
}

__global__ void __launch_bounds__(FB_THREADS, 1)
fused_block_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_we,
                   const __grid_constant__ CUtensorMap tm_wp, const BlockParams p) {
    extern __shared__ uint8_t smem_raw[];
    pdl_trigger();
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - raw);
    // shared-memory map (every part a multiple of 1024 bytes)
    const uint32_t xs_bytes = (uint32_t)(p.cblks * p.MB) * 16384u;
    const uint32_t we_bytes = (uint32_t)p.cblks * 8192u;
    const uint32_t wp_bytes = (uint32_t)p.k_alloc * 128u;                      // k_alloc is a multiple of 16
    const uint32_t h1_bytes = (((uint32_t)((p.H + 2) * (p.W + 2)) * 128u) + 1023u) & ~1023u;
    const uint32_t xs0 = base, we0 = xs0 + xs_bytes, wp0 = we0 + we_bytes;
    const uint32_t wp_end = (wp0 + wp_bytes + 1023u) & ~1023u;
    const uint32_t h1_0 = wp_end, h2_0 = h1_0 + h1_bytes;
    const uint32_t const0 = h2_0 + (uint32_t)p.MB * 16384u;      // this CTA's chunks: [chunk][9 taps x 64 bf16 | 64 be | 64 bd]
    const int my_chunks = (p.nchunks - (int)(blockIdx.x % (unsigned)p.splits) + p.splits - 1) / p.splits;
    const uint32_t ctrl0 = (const0 + (uint32_t)my_chunks * 1664u + 1023u) & ~1023u;
    uint8_t *xs = smem + (xs0 - base), *h1 = smem + (h1_0 - base), *h2 = smem + (h2_0 - base);
    uint8_t *ctrl = smem + (ctrl0 - base);
    const uint32_t bar_x = ctrl0, bar_we = ctrl0 + 8, bar_wp = ctrl0 + 16, bar_m1 = ctrl0 + 24, bar_m2 = ctrl0 + 32;
    uint32_t *tmem_slot = (uint32_t *)(ctrl + 40);
    volatile int *abort_flag = (volatile int *)(ctrl + 44);

    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
    const int n = blockIdx.x / p.splits, rank = blockIdx.x - n * p.splits;
    uint8_t *consts = smem + (const0 - base);

    if (tid == 0) {
        mbar_init(bar_x, 1); mbar_init(bar_we, 1); mbar_init(bar_wp, 1); mbar_init(bar_m1, 1); mbar_init(bar_m2, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_x) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_we) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_wp) : "memory");
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    // the border of the expanded image is the depthwise layer's zero padding: cleared once, only the interior is rewritten
    for (uint32_t e = tid; e < h1_bytes / 16; e += FB_THREADS) ((uint4 *)h1)[e] = make_uint4(0u, 0u, 0u, 0u);
    // depthwise taps and the two hidden-layer biases of this CTA's chunks (written when the block was packed, not by the
    // preceding kernel): once into shared memory, so that no phase of a chunk waits for global memory
    for (int e = tid; e < my_chunks * 104; e += FB_THREADS) {        // 16-byte pieces: 72 of taps, 16 + 16 of biases
        const int it = e / 104, q = e - it * 104;
        const int hch = rank + it * p.splits;                        // chunk number
        uint4 v;
        if (q < 72) v = __ldg((const uint4 *)(p.wd + (size_t)(q >> 3) * (p.hid_alloc >> 3) + hch * 8 + (q & 7)));
        else if (q < 88) v = __ldg((const uint4 *)(p.be + hch * FB_CHUNK) + (q - 72));
        else v = __ldg((const uint4 *)(p.bd + hch * FB_CHUNK) + (q - 88));
        *(uint4 *)(consts + (size_t)it * 1664 + q * 16) = v;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t acc2_col = (uint32_t)(p.MB * FB_CHUNK);

    if (tid == 0) {
        // filters do not depend on the preceding kernel; the image does
        mbar_expect_tx(bar_we, we_bytes);
        for (int cb = 0; cb < p.cblks; ++cb) tma_load_2d(we0 + (uint32_t)cb * 8192u, &tm_we, bar_we, cb * 64, rank * FB_CHUNK);
        mbar_expect_tx(bar_wp, wp_bytes);
        tma_load_2d(wp0, &tm_wp, bar_wp, rank * FB_CHUNK, 0);
        pdl_wait();
        mbar_expect_tx(bar_x, (uint32_t)(p.cblks * p.HW) * 128u);
        for (int cb = 0; cb < p.cblks; ++cb) tma_load_2d(xs0 + (uint32_t)(cb * p.MB) * 16384u, &tm_x, bar_x, cb * 64, n * p.HW);
    }

    // ---- per-thread constants
    // accumulator rows: a warp reads the 32 tensor-memory lanes of its quarter; `part` picks 16 of a chunk's 64 columns
    const int quarter = warp & 3, part = warp >> 2;
    const int row = quarter * 32 + lane;
    const int Wb = p.W + 2;
    int pix1[2];                               // position of this thread's pixel of block mb in the bordered image, or -1
#pragma unroll
    for (int mb = 0; mb < 2; ++mb) {
        const int px = mb * 128 + row;
        pix1[mb] = -1;
        if (mb < p.MB && px < p.HW) { const int i = px / p.W; pix1[mb] = (i + 1) * Wb + (px - i * p.W) + 1; }
    }
    // depthwise: a thread owns channel group g (8 channels) of a run of up to 8 neighbouring pixels of one image row, so that
    // every value of the expanded image is read and unpacked once per filter row instead of once per tap
    const int g = tid & 7;
    const int run_len = p.W <= 8 ? p.W : (p.W + 1) / 2;             // W <= 16 (the bordered image fits 256 pixels)
    const int runs_per_row = (p.W + run_len - 1) / run_len;
    const int dw_run = tid >> 3;                                     // run number; 64 runs cover 14 rows x 2 runs and more
    const int dw_i = dw_run / runs_per_row, dw_j0 = (dw_run - dw_i * runs_per_row) * run_len;
    const bool dw_active = dw_i < p.H;
    const int dw_n = dw_active ? min(run_len, p.W - dw_j0) : 0;      // outputs of this thread
    const uint32_t idesc1 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(FB_CHUNK >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
    const uint32_t idesc2 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.k_alloc >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);

    bool ok = true;
    for (int h = 0; h < my_chunks && ok; ++h) {          // h counts this CTA's chunks; the chunk itself is rank + h * splits
        const uint32_t par = (uint32_t)(h & 1);
        const int hch = rank + h * p.splits;
        // ------------------------------------------------------------ expand MMAs
        if (tid == 0) {
            bool w = h > 0 || mbar_wait(bar_x, 0u, abort_flag, p.status);
            w = w && mbar_wait(bar_we, par, abort_flag, p.status);
            if (w) {
                tc_fence_after();
                for (int mb = 0; mb < p.MB; ++mb) {
                    uint32_t accumulate = 0;
                    for (int cb = 0; cb < p.cblks; ++cb) {
                        const uint64_t da = smem_desc_sw128(xs0 + (uint32_t)(cb * p.MB + mb) * 16384u);
                        const uint64_t db = smem_desc_sw128(we0 + (uint32_t)cb * 8192u);
                        const int nk = cb == p.cblks - 1 ? p.nk_last : 4;
                        for (int kk = 0; kk < nk; ++kk) {
                            umma_bf16(tmem_base + (uint32_t)(mb * FB_CHUNK), da + (uint64_t)(2 * kk), db + (uint64_t)(2 * kk), idesc1, accumulate);
                            accumulate = 1;
                        }
                    }
                }
                umma_commit(bar_m1);
            }
        }
        ok = mbar_wait(bar_m1, par, abort_flag, p.status);
        ok = __syncthreads_and(ok);
        if (!ok) break;
        tc_fence_after();
        if (tid == 0 && h + 1 < my_chunks) {          // the expand filters of the next chunk (their buffer was just read)
            mbar_expect_tx(bar_we, we_bytes);
            for (int cb = 0; cb < p.cblks; ++cb) tma_load_2d(we0 + (uint32_t)cb * 8192u, &tm_we, bar_we, cb * 64, (hch + p.splits) * FB_CHUNK);
        }
        // ------------------------------------------------------------ stage 1: acc1 -> bordered bf16 image
        {
            const float *be = (const float *)(consts + (size_t)h * 1664 + 1152) + part * 16;
            float bias[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) bias[j] = be[j];
            for (int mb = 0; mb < p.MB; ++mb) {
                uint32_t v[16];
                tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(mb * FB_CHUNK + part * 16), v);
                tmem_ld_wait();
                const int pos = mb == 0 ? pix1[0] : pix1[1];
                if (pos >= 0) {
                    float f[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) f[j] = act_apply(__uint_as_float(v[j]) + bias[j], p.act);
                    uint8_t *px = h1 + (size_t)pos * 128;
                    *(bf16x8 *)(px + (((part * 2) ^ (pos & 7)) << 4)) = pack8(f);
                    *(bf16x8 *)(px + (((part * 2 + 1) ^ (pos & 7)) << 4)) = pack8(f + 8);
                }
            }
        }
        tc_fence_before();
        // the depthwise phase overwrites H2, which the project MMAs of the previous chunk read
        if (h > 0) ok = mbar_wait(bar_m2, par ^ 1u, abort_flag, p.status);
        ok = __syncthreads_and(ok);
        if (!ok) break;
        if (tid == 0 && h > 0) {                      // ... and their filters, whose buffer is free now
            mbar_expect_tx(bar_wp, wp_bytes);
            tma_load_2d(wp0, &tm_wp, bar_wp, hch * FB_CHUNK, 0);
        }
        // ------------------------------------------------------------ depthwise 3x3 on the CUDA cores
        {
            const uint8_t *cc = consts + (size_t)h * 1664;
            if (dw_n > 0) {
                float acc[8][8];
#pragma unroll
                for (int o = 0; o < 8; ++o)
#pragma unroll
                    for (int i = 0; i < 8; ++i) acc[o][i] = ((const float *)(cc + 1408))[g * 8 + i];
#pragma unroll
                for (int r = 0; r < 3; ++r) {
                    float wf[3][8];
#pragma unroll
                    for (int t = 0; t < 3; ++t) unpack8(*(const bf16x8 *)(cc + ((r * 3 + t) * 8 + g) * 16), wf[t]);
                    const int pos0 = (dw_i + r) * Wb + dw_j0;       // bordered-image position left of the run's first pixel, row r
#pragma unroll
                    for (int sx = 0; sx < 10; ++sx) {
                        if (sx < dw_n + 2) {
                            const int pos = pos0 + sx;
                            float xf[8];
                            unpack8(*(const bf16x8 *)(h1 + (size_t)pos * 128 + ((g ^ (pos & 7)) << 4)), xf);
#pragma unroll
                            for (int t = 0; t < 3; ++t) {
                                const int o = sx - t;                // output this value feeds through tap column t
                                if (o >= 0 && o < 8) {
#pragma unroll
                                    for (int i = 0; i < 8; ++i) acc[o][i] = fmaf(xf[i], wf[t][i], acc[o][i]);
                                }
                            }
                        }
                    }
                }
#pragma unroll
                for (int o = 0; o < 8; ++o) {
                    if (o < dw_n) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) acc[o][i] = act_apply(acc[o][i], p.act);
                        const int px = dw_i * p.W + dw_j0 + o;
                        *(bf16x8 *)(h2 + (size_t)(px >> 7) * 16384 + sub_off(px & 127, g)) = pack8(acc[o]);
                    }
                }
            }
        }
        fence_async_smem();                           // H2 was written by ordinary stores and is read by the tensor core
        __syncthreads();
        // ------------------------------------------------------------ project MMAs (run while the next chunk expands)
        if (tid == 0) {
            if (mbar_wait(bar_wp, par, abort_flag, p.status)) {
                tc_fence_after();
                const uint64_t db = smem_desc_sw128(wp0);
                for (int mb = 0; mb < p.MB; ++mb) {
                    const uint64_t da = smem_desc_sw128(h2_0 + (uint32_t)mb * 16384u);
                    for (int kk = 0; kk < 4; ++kk)
                        umma_bf16(tmem_base + acc2_col + (uint32_t)(mb * p.k_alloc), da + (uint64_t)(2 * kk), db + (uint64_t)(2 * kk), idesc2,
                                  (h > 0 || kk > 0) ? 1u : 0u);
                }
                umma_commit(bar_m2);
            }
        }
    }
    // ---------------------------------------------------------------- last phase: bias, residual, store
    if (ok && my_chunks > 0) ok = mbar_wait(bar_m2, (uint32_t)((my_chunks - 1) & 1), abort_flag, p.status);
    ok = __syncthreads_and(ok);
    const int k8 = p.k_pad >> 3;
    uint8_t *stage = h1;                              // H1 and H2 together hold an image's output
    if (ok && p.splits > 1) {
        // this CTA's share of the project sums, float32, for the finalize kernel
        tc_fence_after();
        float *part_out = p.partial + ((size_t)rank * (size_t)p.M + (size_t)n * p.HW) * p.k_alloc;
        for (int mb = 0; mb < p.MB; ++mb) {
            const int px = mb * 128 + row;
            for (int c0 = part * 16; c0 < p.k_alloc; c0 += 64) {
                uint32_t v[16];
                tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + acc2_col + (uint32_t)(mb * p.k_alloc + c0), v);
                tmem_ld_wait();
                if (px < p.HW) {
                    float4 *dst = (float4 *)(part_out + (size_t)px * p.k_alloc + c0);
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        dst[j] = my_chunks > 0 ? make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]), __uint_as_float(v[4 * j + 2]),
                                                             __uint_as_float(v[4 * j + 3]))
                                               : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
        }
    } else if (ok) {
        tc_fence_after();
        for (int mb = 0; mb < p.MB; ++mb) {
            const int px = mb * 128 + row;
            for (int c0 = part * 16; c0 < p.k_alloc; c0 += 64) {
                uint32_t v[16];
                tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + acc2_col + (uint32_t)(mb * p.k_alloc + c0), v);
                tmem_ld_wait();
                if (px < p.HW && c0 < p.k_pad) {
                    float f[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) f[j] = __uint_as_float(v[j]) + __ldg(p.bp + c0 + j);
                    if (p.residual) {
                        const uint8_t *xr = xs + (size_t)((c0 >> 6) * p.MB + mb) * 16384;
                        float rf[8];
                        unpack8(*(const bf16x8 *)(xr + sub_off(row, (c0 & 63) >> 3)), rf);
#pragma unroll
                        for (int j = 0; j < 8; ++j) f[j] += rf[j];
                        unpack8(*(const bf16x8 *)(xr + sub_off(row, ((c0 & 63) >> 3) + 1)), rf);
#pragma unroll
                        for (int j = 0; j < 8; ++j) f[8 + j] += rf[j];
                    }
#pragma unroll
                    for (int j = 0; j < 16; ++j) f[j] = act_apply(f[j], p.act_out);
                    // staged densely ([pixel][k_pad]) with the 16-byte pieces of a pixel rotated by the pixel number, so that
                    // the threads of a warp (neighbouring pixels, same filters) fall into different banks
                    const int c8 = c0 >> 3;
                    *(bf16x8 *)(stage + ((size_t)px * k8 + (c8 + px) % k8) * 16) = pack8(f);
                    if (c8 + 1 < k8) *(bf16x8 *)(stage + ((size_t)px * k8 + (c8 + 1 + px) % k8) * 16) = pack8(f + 8);
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (ok && p.splits == 1) {
        bf16x8 *yimg = p.y + (size_t)n * p.HW * k8;
        for (int e = tid; e < p.HW * k8; e += FB_THREADS) {
            const int px = e / k8, c8 = e - px * k8;
            yimg[e] = *(const bf16x8 *)(stage + ((size_t)px * k8 + (c8 + px) % k8) * 16);
        }
    }
    if (*abort_flag) {
        for (int i = 0; i < 200; ++i) __nanosleep(1000);   // let copies in flight land before the memory goes away
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// ---------------------------------------------------------------------------------------------- packing

// expand [hidden][C_in] -> bf16 [hid_alloc][c_in_pad]; depthwise [hidden][3][3] -> bf16 [9][hid_alloc];
// project [C_out][hidden] -> bf16 [k_alloc][hid_alloc]; zero padded
__global__ void block_pack_kernel(const float *__restrict__ we, const float *__restrict__ wd, const float *__restrict__ wp, int C_in,
                                  int hidden, int C_out, int c_in_pad, int hid_alloc, int k_alloc, __nv_bfloat16 *__restrict__ out) {
    const size_t n_e = (size_t)hid_alloc * c_in_pad, n_d = (size_t)9 * hid_alloc, n_p = (size_t)k_alloc * hid_alloc;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n_e + n_d + n_p; e += (size_t)gridDim.x * blockDim.x) {
        float v = 0.f;
        if (e < n_e) {
            const int hh = (int)(e / c_in_pad), c = (int)(e % c_in_pad);
            if (hh < hidden && c < C_in) v = we[(size_t)hh * C_in + c];
        } else if (e < n_e + n_d) {
            const size_t t = e - n_e;
            const int tap = (int)(t / hid_alloc), hh = (int)(t % hid_alloc);
            if (hh < hidden) v = wd[(size_t)hh * 9 + tap];
        } else {
            const size_t t = e - n_e - n_d;
            const int k = (int)(t / hid_alloc), hh = (int)(t % hid_alloc);
            if (k < C_out && hh < hidden) v = wp[(size_t)k * hidden + hh];
        }
        out[e] = __float2bfloat16_rn(v);
    }
}

__global__ void block_bias_kernel(const float *__restrict__ be, const float *__restrict__ bd, const float *__restrict__ bp, int hidden,
                                  int C_out, int hid_alloc, int k_alloc, float *__restrict__ out) {
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= 2 * hid_alloc + k_alloc) return;
    float v = 0.f;
    if (e < hid_alloc) { if (be && e < hidden) v = be[e]; }
    else if (e < 2 * hid_alloc) { if (bd && e - hid_alloc < hidden) v = bd[e - hid_alloc]; }
    else { if (bp && e - 2 * hid_alloc < C_out) v = bp[e - 2 * hid_alloc]; }
    out[e] = v;
}

}  // namespace cprune

// ---------------------------------------------------------------------------------------------- host

using namespace cprune;

namespace {

struct BlockCache {
    std::mutex mu;
    std::map<std::array<int, 9>, cprune_block *> blocks;
};
BlockCache &block_cache() {
    static BlockCache c;
    return c;
}

}  // namespace

extern "C" {

cprune_status cprune_block_plan(int N, int C_in, int H, int W, int hidden, int C_out, int act, int act_out, int residual,
                                cprune_block **out) {
    if (!out) return CPRUNE_ERR_INVALID_ARG;
    *out = nullptr;
    if (N <= 0 || C_in <= 0 || H <= 0 || W <= 0 || hidden <= 0 || C_out <= 0 || act < 0 || act > 2 || act_out < 0 || act_out > 2 ||
        (residual != 0 && residual != 1))
        return CPRUNE_ERR_INVALID_ARG;
    if (residual && C_in != C_out) return CPRUNE_ERR_INVALID_ARG;
    const int HW = H * W, MB = (HW + 127) / 128;
    const int c_in_pad = cprune_padded_channels(C_in), k_pad = cprune_padded_channels(C_out);
    const int k_alloc = round_up(C_out, 16), hid_alloc = round_up(hidden, FB_CHUNK), cblks = (c_in_pad + 63) / 64;
    // one CTA holds an image: pixels within two accumulator blocks, the bordered expanded image within 32 KB, filters within one
    // MMA, accumulators within tensor memory, the staged output within the two hidden-tensor buffers
    if (HW > 256 || (H + 2) * (W + 2) > 256 || cblks > 3 || k_alloc > 256) return CPRUNE_ERR_UNSUPPORTED;
    // depthwise phase: a thread takes a run of at most 8 pixels of a row, 64 runs per channel group
    if (W > 16 || H * ((W + (W <= 8 ? W : (W + 1) / 2) - 1) / (W <= 8 ? W : (W + 1) / 2)) > FB_THREADS / 8) return CPRUNE_ERR_UNSUPPORTED;
    if (MB * (FB_CHUNK + k_alloc) > 512) return CPRUNE_ERR_UNSUPPORTED;
    const int h1_bytes = round_up((H + 2) * (W + 2) * 128, 1024);
    if ((size_t)HW * k_pad * 2 > (size_t)h1_bytes + (size_t)MB * 16384) return CPRUNE_ERR_UNSUPPORTED;
    // CTAs per image: a block's time is a chain of about 3 us per 64-channel chunk plus about 4 us of set-up and drain; the chunks
    // of an image are dealt to `splits` CTAs when that shortens the chain by more than the second pass (about 4 us) costs
    const int nchunks = hid_alloc / FB_CHUNK;
    int splits = 1;
    double best = 1e30;
    for (int sp = 1; sp <= nchunks && sp <= 16; ++sp) {
        const int per = (nchunks + sp - 1) / sp;
        if ((sp - 1) * per >= nchunks) continue;                  // a CTA would be left without a chunk
        const double waves = (double)(((long long)N * sp + 147) / 148);
        const double t = waves * (per * 3.0 + 4.0) + (sp > 1 ? 4.0 : 0.0);
        if (t < best - 1e-9) { best = t; splits = sp; }
    }
    const int per_cta = (nchunks + splits - 1) / splits;
    const int smem = 1024 + cblks * MB * 16384 + cblks * 8192 + round_up(k_alloc * 128, 1024) + h1_bytes + MB * 16384 +
                     round_up(per_cta * 1664, 1024) + 1024;
    if (smem > 227 * 1024) return CPRUNE_ERR_UNSUPPORTED;
    if ((long long)N * HW > 0x7fffffffLL) return CPRUNE_ERR_UNSUPPORTED;
    std::array<int, 9> key = {N, C_in, H, W, hidden, C_out, act, act_out, residual};
    BlockCache &c = block_cache();
    std::lock_guard<std::mutex> lock(c.mu);
    auto it = c.blocks.find(key);
    if (it != c.blocks.end()) {
        ++it->second->refs;
        *out = it->second;
        return CPRUNE_OK;
    }
    cprune_block *b = new cprune_block();
    cprune_block_info &i = b->info;
    i = cprune_block_info();
    i.N = N; i.C_in = C_in; i.H = H; i.W = W; i.hidden = hidden; i.C_out = C_out; i.act = act; i.act_out = act_out; i.residual = residual;
    i.c_in_pad = c_in_pad; i.k_pad = k_pad; i.hid_alloc = hid_alloc; i.k_alloc = k_alloc;
    i.packed_weight_bytes = ((size_t)hid_alloc * c_in_pad + (size_t)9 * hid_alloc + (size_t)k_alloc * hid_alloc) * 2;
    i.packed_bias_bytes = ((size_t)2 * hid_alloc + k_alloc) * sizeof(float);
    i.flops = 2.0 * N * HW * ((double)C_in * hidden + 9.0 * hidden + (double)hidden * C_out);
    const double weights = 2.0 * ((double)C_in * hidden + 9.0 * hidden + (double)hidden * C_out) + 4.0 * (2.0 * hidden + C_out);
    i.algorithmic_bytes = 2.0 * N * HW * ((double)C_in + C_out) + weights;                    // the residual is the input: read once
    i.unfused_bytes = i.algorithmic_bytes + 2.0 * N * HW * 4.0 * hidden + (residual ? 2.0 * N * HW * C_in : 0.0);
    b->MB = MB; b->cblks = cblks; b->nk_last = (c_in_pad - (cblks - 1) * 64 + 15) / 16; b->nchunks = nchunks;
    b->smem_bytes = smem;
    b->splits = splits;
    i.splits = splits;
    i.workspace_bytes = splits > 1 ? (size_t)splits * N * HW * k_alloc * sizeof(float) : 0;
    i.est_us = best;
    b->refs = 1;
    c.blocks[key] = b;
    *out = b;
    return CPRUNE_OK;
}

cprune_status cprune_block_query(const cprune_block *block, cprune_block_info *out) {
    if (!block || !out) return CPRUNE_ERR_INVALID_ARG;
    *out = block->info;
    return CPRUNE_OK;
}

cprune_status cprune_block_release(cprune_block *block) {
    if (!block) return CPRUNE_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(block_cache().mu);
    if (block->refs <= 0) return CPRUNE_ERR_INVALID_ARG;
    --block->refs;
    return CPRUNE_OK;
}

cprune_status cprune_block_pack(const cprune_block *block, const float *w_expand, const float *b_expand, const float *w_depthwise,
                                const float *b_depthwise, const float *w_project, const float *b_project, void *w_packed,
                                float *b_packed, void *stream) {
    if (!block || !w_expand || !w_depthwise || !w_project || !w_packed || !b_packed) return CPRUNE_ERR_INVALID_ARG;
    const cprune_block_info &i = block->info;
    const size_t total = i.packed_weight_bytes / 2;
    size_t blocks = (total + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    block_pack_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(w_expand, w_depthwise, w_project, i.C_in, i.hidden, i.C_out,
                                                                         i.c_in_pad, i.hid_alloc, i.k_alloc, (__nv_bfloat16 *)w_packed);
    CPRUNE_LAUNCH_CHECK("block_pack_kernel");
    const int nb = 2 * i.hid_alloc + i.k_alloc;
    block_bias_kernel<<<(nb + 255) / 256, 256, 0, (cudaStream_t)stream>>>(b_expand, b_depthwise, b_project, i.hidden, i.C_out, i.hid_alloc,
                                                                         i.k_alloc, b_packed);
    CPRUNE_LAUNCH_CHECK("block_bias_kernel");
    return CPRUNE_OK;
}

cprune_status cprune_block_run(cprune_block *block, const void *x, const void *w_packed, const float *b_packed, void *y, void *workspace,
                               void *stream) {
    if (!block || !x || !w_packed || !b_packed || !y) return CPRUNE_ERR_INVALID_ARG;
    if (((uintptr_t)x | (uintptr_t)w_packed | (uintptr_t)y | (uintptr_t)workspace) & 15) return CPRUNE_ERR_INVALID_ARG;
    if (block->info.workspace_bytes && !workspace) return CPRUNE_ERR_INVALID_ARG;
    const cprune_block_info &i = block->info;
    const int HW = i.H * i.W;
    const __nv_bfloat16 *wq = (const __nv_bfloat16 *)w_packed;
    const __nv_bfloat16 *we = wq, *wd = wq + (size_t)i.hid_alloc * i.c_in_pad, *wp = wd + (size_t)9 * i.hid_alloc;
    CUtensorMap tm_x, tm_we, tm_wp;
    {
        std::lock_guard<std::mutex> lock(block->mu);
        if (block->map_x != x) {
            const unsigned long long dims[2] = {(unsigned long long)i.c_in_pad, (unsigned long long)i.N * HW};
            const unsigned long long strides[1] = {(unsigned long long)i.c_in_pad * 2};
            const unsigned box[2] = {64, (unsigned)HW};
            cprune_status s = encode_tiled_bf16_swz(&block->tm_x, x, 2, dims, strides, box, 128, true);
            if (s != CPRUNE_OK) return s;
            block->map_x = x;
        }
        if (block->map_w != w_packed) {
            const unsigned long long de[2] = {(unsigned long long)i.c_in_pad, (unsigned long long)i.hid_alloc};
            const unsigned long long se[1] = {(unsigned long long)i.c_in_pad * 2};
            const unsigned be[2] = {64, (unsigned)FB_CHUNK};
            cprune_status s = encode_tiled_bf16_swz(&block->tm_we, we, 2, de, se, be, 128, true);
            if (s != CPRUNE_OK) return s;
            const unsigned long long dp[2] = {(unsigned long long)i.hid_alloc, (unsigned long long)i.k_alloc};
            const unsigned long long sp[1] = {(unsigned long long)i.hid_alloc * 2};
            const unsigned bp[2] = {64, (unsigned)i.k_alloc};
            s = encode_tiled_bf16_swz(&block->tm_wp, wp, 2, dp, sp, bp, 128, true);
            if (s != CPRUNE_OK) return s;
            block->map_w = w_packed;
        }
        std::memcpy(&tm_x, &block->tm_x, sizeof(CUtensorMap));
        std::memcpy(&tm_we, &block->tm_we, sizeof(CUtensorMap));
        std::memcpy(&tm_wp, &block->tm_wp, sizeof(CUtensorMap));
    }
    static std::mutex attr_mu;
    static bool attr_set[64] = {false};
    {
        int dev = 0;
        CPRUNE_CUDA_CHECK(cudaGetDevice(&dev));
        if (dev < 0 || dev >= 64) return CPRUNE_ERR_UNSUPPORTED;
        std::lock_guard<std::mutex> lock(attr_mu);
        if (!attr_set[dev]) {
            CPRUNE_CUDA_CHECK(cudaFuncSetAttribute(fused_block_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            attr_set[dev] = true;
        }
    }
    BlockParams p;
    p.HW = HW; p.H = i.H; p.W = i.W; p.MB = block->MB; p.cblks = block->cblks; p.nk_last = block->nk_last; p.nchunks = block->nchunks;
    p.hid_alloc = i.hid_alloc; p.k_alloc = i.k_alloc; p.k_pad = i.k_pad; p.act = i.act; p.act_out = i.act_out; p.residual = i.residual;
    p.be = b_packed; p.bd = b_packed + i.hid_alloc; p.bp = b_packed + 2 * i.hid_alloc;
    p.wd = (const bf16x8 *)wd;
    p.y = (bf16x8 *)y;
    p.splits = block->splits;
    p.partial = (float *)workspace;
    p.M = (long long)i.N * HW;
    p.status = device_status_word();
    if (!p.status) return cuda_fail(cudaGetLastError(), "status word");
    CPRUNE_CUDA_CHECK(launch_chained(fused_block_kernel, dim3((unsigned)(i.N * block->splits)), dim3(FB_THREADS), (size_t)block->smem_bytes,
                                     (cudaStream_t)stream, tm_x, tm_we, tm_wp, p));
    if (block->splits > 1)
        return launch_splitk_finalize((const float *)workspace, block->splits, p.M, i.k_alloc, i.k_pad, p.bp, i.residual ? x : nullptr,
                                      i.act_out, y, (cudaStream_t)stream);
    return CPRUNE_OK;
}

}  // extern "C"
