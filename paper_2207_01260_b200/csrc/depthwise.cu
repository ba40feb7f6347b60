// Depthwise task (groups == C == K), 3x3 or 5x5 (MobileNetV2 and MnasNet, paper Sec. 4.1): memory-bound, CUDA
// cores.  bf16 NHWC in and out with padded channels, float32 arithmetic, fused bias + activation (+ residual).
//
// One CTA computes TH x TW output pixels of one image for one block of 64 channels.  Its input
// patch ((TH-1)*stride+3) x ((TW-1)*stride+3) pixels x 64 channels comes in with a single tiled
// TMA load (out-of-bounds pixels and channels read as zero, which is the padding), so every input
// byte is fetched from L2/HBM once per CTA and the nine taps are served from shared memory.
// A thread owns 8 channels of one output column and walks down the TH rows; threads of a warp
// cover the 8 channel groups of 4 neighbouring columns, i.e. four contiguous 128-byte pixels.
// Several CTAs share an SM, so one CTA's load overlaps the arithmetic of the others.  The wait
// on the load is bounded like every other device-side wait of the library.
#include <cstring>

#include "common.cuh"
#include "plan.h"

namespace cprune {

struct DwParams {
    const bf16x8 *w;   // [3][3][c8]
    const float *b;
    const bf16x8 *res;
    bf16x8 *y;
    int P, Q, pad, act, R;
    int c8;            // c_pad / 8
    int G;             // channel groups (of 8) per CTA: min(8, c8)
    int TH, TW, IH, IW;
    int tiles_h, tiles_w, cblocks;
    int *status;
};

__device__ __forceinline__ uint32_t dw_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// a0 += x.lo * w.lo, a1 += x.hi * w.hi for two packed bf16 pairs: the mixed-precision fused multiply-add takes bf16
// factors and a float32 addend.  A product of two bf16 values is exact in float32, so the result is the one
// fmaf(float(x), float(w), a) gives, without the two conversions per pair.
__device__ __forceinline__ void fma_bf16x2(float &a0, float &a1, uint32_t x, uint32_t w) {
    asm("{\n\t"
        ".reg .b16 xl, xh, wl, wh;\n\t"
        "mov.b32 {xl, xh}, %2;\n\t"
        "mov.b32 {wl, wh}, %3;\n\t"
        "fma.rn.f32.bf16 %0, xl, wl, %0;\n\t"
        "fma.rn.f32.bf16 %1, xh, wh, %1;\n\t"
        "}"
        : "+f"(a0), "+f"(a1)
        : "r"(x), "r"(w));
}

template <int STRIDE>
__global__ void __launch_bounds__(256) depthwise3x3_kernel(const __grid_constant__ CUtensorMap tm_x, const DwParams p) {
    extern __shared__ __align__(128) uint8_t dw_smem[];
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int failed;

    pdl_trigger();
    pdl_wait();
    int bid = blockIdx.x;
    const int cb = bid % p.cblocks; bid /= p.cblocks;
    const int tw = bid % p.tiles_w; bid /= p.tiles_w;
    const int th = bid % p.tiles_h;
    const int n = bid / p.tiles_h;
    const int p0 = th * p.TH, q0 = tw * p.TW;
    const int G = p.G;

    const uint32_t bar_a = dw_smem_u32(&bar);
    if (threadIdx.x == 0) {
        failed = 0;
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_a) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const uint32_t bytes = (uint32_t)(p.IH * p.IW * G * 16);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_a), "r"(bytes) : "memory");
        asm volatile(
            "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
            :
            : "r"(dw_smem_u32(dw_smem)), "l"(&tm_x), "r"(bar_a), "r"(cb * G * 8), "r"(q0 * STRIDE - p.pad),
              "r"(p0 * STRIDE - p.pad), "r"(n)
            : "memory");
    }
    __syncthreads();   // the barrier is initialised before anyone polls it

    const int cg = threadIdx.x % G;          // channel group within the CTA's channel block
    const int qq = threadIdx.x / G;          // output column within the tile
    const int cgg = cb * G + cg;             // channel group within the tensor
    const bool active = qq < p.TW && q0 + qq < p.Q && cgg < p.c8;

    // filter taps (bf16 pairs, as packed) and bias of this thread's 8 channels (overlaps the load)
    bf16x8 wq[9];
    float bf[8];
    if (active) {
#pragma unroll
        for (int t = 0; t < 9; ++t) wq[t] = ldg8(p.w + (size_t)t * p.c8 + cgg);
#pragma unroll
        for (int i = 0; i < 8; ++i) bf[i] = __ldg(p.b + cgg * 8 + i);
    }

    // bounded wait for the patch
    {
        uint32_t ok = 0;
        long long t0 = clock64();
        while (true) {
            asm volatile(
                "{\n\t.reg .pred q;\n\t"
                "mbarrier.try_wait.parity.shared::cta.b64 q, [%1], 0;\n\t"
                "selp.u32 %0, 1, 0, q;\n\t}"
                : "=r"(ok)
                : "r"(bar_a)
                : "memory");
            if (ok) break;
            if (clock64() - t0 > (1LL << 31)) {
                atomicOr(p.status, STATUS_TIMEOUT);
                failed = 1;
                break;
            }
        }
    }
    __syncthreads();
    if (failed) {
        for (int i = 0; i < 200; ++i) __nanosleep(1000);   // let a late copy land before the CTA's memory goes away
        return;
    }
    if (!active) return;

    const bf16x8 *patch = reinterpret_cast<const bf16x8 *>(dw_smem) + cg;   // [IH][IW][G groups]
    const size_t out_row = (size_t)p.Q * p.c8;
    const size_t o0 = (((size_t)n * p.P + p0) * p.Q + q0 + qq) * p.c8 + cgg;

    auto finish = [&](float *acc, int pp) {
        const size_t o = o0 + (size_t)pp * out_row;
        if (p.res) {
            float rf[8];
            unpack8(ldg8(p.res + o), rf);
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] += rf[i];
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = apply_act(acc[i], p.act);
        p.y[o] = pack8(acc);
    };

    if (STRIDE == 1) {
        // walk down the input rows; each row feeds the three output rows it overlaps.  An input value is used three
        // times here, so it is converted to float32 once (measured: faster than the mixed-precision form below, and
        // than packed float32 pairs with rotating accumulators)
        const int rows = min(p.TH, p.P - p0);       // output rows of this tile
        float wf[9][8];
#pragma unroll
        for (int t = 0; t < 9; ++t) unpack8(wq[t], wf[t]);
        float a0[8], a1[8], a2[8];                  // accumulators of output rows h-2, h-1, h
#pragma unroll
        for (int i = 0; i < 8; ++i) { a0[i] = bf[i]; a1[i] = bf[i]; a2[i] = bf[i]; }
        for (int h = 0; h < rows + 2; ++h) {
            const bf16x8 *row = patch + ((size_t)h * p.IW + qq) * G;
            float x[3][8];
#pragma unroll
            for (int s = 0; s < 3; ++s) unpack8(row[s * G], x[s]);
#pragma unroll
            for (int s = 0; s < 3; ++s)
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    a0[i] = fmaf(x[s][i], wf[6 + s][i], a0[i]);   // this row is tap row 2 of output row h-2
                    a1[i] = fmaf(x[s][i], wf[3 + s][i], a1[i]);   // tap row 1 of output row h-1
                    a2[i] = fmaf(x[s][i], wf[s][i], a2[i]);       // tap row 0 of output row h
                }
            if (h >= 2) finish(a0, h - 2);
#pragma unroll
            for (int i = 0; i < 8; ++i) { a0[i] = a1[i]; a1[i] = a2[i]; a2[i] = bf[i]; }
        }
    } else {
        // an input value is used once per output row here: the mixed-precision FMA saves its conversion
        for (int pp = 0; pp < p.TH && p0 + pp < p.P; ++pp) {
            float acc[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] = bf[i];
#pragma unroll
            for (int r = 0; r < 3; ++r) {
                const bf16x8 *row = patch + ((size_t)(pp * STRIDE + r) * p.IW + qq * STRIDE) * G;
#pragma unroll
                for (int s = 0; s < 3; ++s) {
                    const bf16x8 x = row[s * G];
#pragma unroll
                    for (int j = 0; j < 4; ++j) fma_bf16x2(acc[2 * j], acc[2 * j + 1], x.w[j], wq[r * 3 + s].w[j]);
                }
            }
            finish(acc, pp);
        }
    }
}

// R x R taps for filters too large to keep in registers (5x5): the same tiling and patch load as above; the CTA's
// filter taps are converted to float32 in shared memory once, and a thread (8 channels of one output column) walks
// down the tile's rows, reading every tap of its window from the patch.
template <int STRIDE, int R>
__global__ void __launch_bounds__(256) depthwise_rxr_kernel(const __grid_constant__ CUtensorMap tm_x, const DwParams p) {
    extern __shared__ __align__(128) uint8_t dw_smem[];
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int failed;
    __shared__ __align__(16) float wsm[R * R][9][8];      // [tap][channel group of the CTA][channel]

    pdl_trigger();
    pdl_wait();
    int bid = blockIdx.x;
    const int cb = bid % p.cblocks; bid /= p.cblocks;
    const int tw = bid % p.tiles_w; bid /= p.tiles_w;
    const int th = bid % p.tiles_h;
    const int n = bid / p.tiles_h;
    const int p0 = th * p.TH, q0 = tw * p.TW;
    const int G = p.G;

    const uint32_t bar_a = dw_smem_u32(&bar);
    if (threadIdx.x == 0) {
        failed = 0;
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_a) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const uint32_t bytes = (uint32_t)(p.IH * p.IW * G * 16);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_a), "r"(bytes) : "memory");
        asm volatile(
            "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
            :
            : "r"(dw_smem_u32(dw_smem)), "l"(&tm_x), "r"(bar_a), "r"(cb * G * 8), "r"(q0 * STRIDE - p.pad),
              "r"(p0 * STRIDE - p.pad), "r"(n)
            : "memory");
    }
    // filter taps of the CTA's channel groups (overlaps the load); groups beyond the tensor read as zero
    for (int e = threadIdx.x; e < R * R * G; e += blockDim.x) {
        const int t = e / G, g = e - t * G;
        float f[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (cb * G + g < p.c8) unpack8(ldg8(p.w + (size_t)t * p.c8 + cb * G + g), f);
#pragma unroll
        for (int i = 0; i < 8; ++i) wsm[t][g][i] = f[i];
    }
    __syncthreads();   // the barrier is initialised and the taps are in place before anyone goes on

    const int cg = threadIdx.x % G;
    const int qq = threadIdx.x / G;
    const int cgg = cb * G + cg;
    const bool active = qq < p.TW && q0 + qq < p.Q && cgg < p.c8;
    float bf[8];
    if (active) {
#pragma unroll
        for (int i = 0; i < 8; ++i) bf[i] = __ldg(p.b + cgg * 8 + i);
    }
    {
        uint32_t ok = 0;
        long long t0 = clock64();
        while (true) {
            asm volatile(
                "{\n\t.reg .pred q;\n\t"
                "mbarrier.try_wait.parity.shared::cta.b64 q, [%1], 0;\n\t"
                "selp.u32 %0, 1, 0, q;\n\t}"
                : "=r"(ok)
                : "r"(bar_a)
                : "memory");
            if (ok) break;
            if (clock64() - t0 > (1LL << 31)) {
                atomicOr(p.status, STATUS_TIMEOUT);
                failed = 1;
                break;
            }
        }
    }
    __syncthreads();
    if (failed) {
        for (int i = 0; i < 200; ++i) __nanosleep(1000);   // let a late copy land before the CTA's memory goes away
        return;
    }
    if (!active) return;

    const bf16x8 *patch = reinterpret_cast<const bf16x8 *>(dw_smem) + cg;   // [IH][IW][G groups]
    const size_t out_row = (size_t)p.Q * p.c8;
    const size_t o0 = (((size_t)n * p.P + p0) * p.Q + q0 + qq) * p.c8 + cgg;
    for (int pp = 0; pp < p.TH && p0 + pp < p.P; ++pp) {
        float acc[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = bf[i];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const bf16x8 *row = patch + ((size_t)(pp * STRIDE + r) * p.IW + qq * STRIDE) * G;
#pragma unroll
            for (int s2 = 0; s2 < R; ++s2) {
                float xf[8];
                unpack8(row[s2 * G], xf);
                const float4 w0 = *reinterpret_cast<const float4 *>(&wsm[r * R + s2][cg][0]);
                const float4 w1 = *reinterpret_cast<const float4 *>(&wsm[r * R + s2][cg][4]);
                acc[0] = fmaf(xf[0], w0.x, acc[0]); acc[1] = fmaf(xf[1], w0.y, acc[1]);
                acc[2] = fmaf(xf[2], w0.z, acc[2]); acc[3] = fmaf(xf[3], w0.w, acc[3]);
                acc[4] = fmaf(xf[4], w1.x, acc[4]); acc[5] = fmaf(xf[5], w1.y, acc[5]);
                acc[6] = fmaf(xf[6], w1.z, acc[6]); acc[7] = fmaf(xf[7], w1.w, acc[7]);
            }
        }
        const size_t o = o0 + (size_t)pp * out_row;
        if (p.res) {
            float rf[8];
            unpack8(ldg8(p.res + o), rf);
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] += rf[i];
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = apply_act(acc[i], p.act);
        p.y[o] = pack8(acc);
    }
}

// Tile of output pixels per CTA and channel groups per CTA.
// Channel groups (of 8 channels) per CTA: between 4 and 9, whichever wastes the fewest lanes in
// the last channel block (c_pad/8 = 18 -> 9, 14 -> 7, 4 -> 4); larger wins ties.
int depthwise_groups(int c8) {
    if (c8 <= 9) return c8;
    int best = 8;
    double best_util = 0.0;
    for (int g = 9; g >= 4; --g) {
        const double util = (double)c8 / (double)(((c8 + g - 1) / g) * g);
        if (util > best_util + 1e-9) { best_util = util; best = g; }
    }
    return best;
}

// Tile of output pixels per CTA and channel groups per CTA.
static void dw_tile(const cprune_plan_info &i, int *TH, int *TW, int *G) {
    const int c8 = i.c_pad / 8;
    *G = depthwise_groups(c8);
    int tw = 112 / *G;                      // about 112 threads per CTA: small patches, several CTAs per SM
    if (i.stride == 2 && tw > 28) tw = 28;  // keeps the input patch small
    *TW = i.Q < tw ? i.Q : tw;
    int th = i.stride == 1 ? 14 : (*TW <= 14 ? 7 : 4);
    if (i.R > 3 && i.stride == 2 && *TW > 14) *TW = 14;      // larger filters: keep the input patch within shared memory
    *TH = i.P < th ? i.P : th;
}

cprune_status launch_depthwise(cprune_plan *plan, const void *x, const void *w, const float *b, const void *res,
                               void *y, cudaStream_t st) {
    const cprune_plan_info &i = plan->info;
    DwParams p;
    p.w = (const bf16x8 *)w;
    p.b = b;
    p.res = (const bf16x8 *)res;
    p.y = (bf16x8 *)y;
    p.P = i.P; p.Q = i.Q; p.pad = i.pad; p.act = plan->opts.activation; p.R = i.R;
    p.c8 = i.c_pad / 8;
    dw_tile(i, &p.TH, &p.TW, &p.G);
    p.IH = (p.TH - 1) * i.stride + i.R;
    p.IW = (p.TW - 1) * i.stride + i.S;
    p.tiles_h = (i.P + p.TH - 1) / p.TH;
    p.tiles_w = (i.Q + p.TW - 1) / p.TW;
    p.cblocks = (p.c8 + p.G - 1) / p.G;
    p.status = device_status_word();
    if (!p.status) return cuda_fail(cudaGetLastError(), "status word");
    CUtensorMap tm;
    {
        std::lock_guard<std::mutex> lock(plan->mu);
        if (plan->map_x != x) {
            unsigned long long dims[4] = {(unsigned long long)i.c_pad, (unsigned long long)i.W, (unsigned long long)i.H,
                                          (unsigned long long)i.N};
            unsigned long long strides[3] = {(unsigned long long)i.c_pad * 2, (unsigned long long)i.W * i.c_pad * 2,
                                             (unsigned long long)i.H * i.W * i.c_pad * 2};
            unsigned box[4] = {(unsigned)(p.G * 8), (unsigned)p.IW, (unsigned)p.IH, 1};
            cprune_status s = encode_tiled_bf16(&plan->tm_a, x, 4, dims, strides, box);
            if (s != CPRUNE_OK) return s;
            plan->map_x = x;
        }
        std::memcpy(&tm, &plan->tm_a, sizeof(CUtensorMap));
    }
    const long long blocks = (long long)i.N * p.tiles_h * p.tiles_w * p.cblocks;
    if (blocks == 0) return CPRUNE_OK;
    if (blocks > 0x7fffffffLL || p.IW > 256 || p.IH > 256) return CPRUNE_ERR_UNSUPPORTED;
    const int smem = p.IH * p.IW * p.G * 16;
    static std::mutex attr_mu;
    static int attr_set[64] = {0};     // the shared-memory limit of a kernel is a per-device attribute
    {
        int dev = 0;
        CPRUNE_CUDA_CHECK(cudaGetDevice(&dev));
        if (dev < 0 || dev >= 64) return CPRUNE_ERR_UNSUPPORTED;
        std::lock_guard<std::mutex> lock(attr_mu);
        if (!attr_set[dev]) {
            CPRUNE_CUDA_CHECK(cudaFuncSetAttribute(depthwise3x3_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024));
            CPRUNE_CUDA_CHECK(cudaFuncSetAttribute(depthwise3x3_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024));
            CPRUNE_CUDA_CHECK(cudaFuncSetAttribute(depthwise_rxr_kernel<1, 5>, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024));
            CPRUNE_CUDA_CHECK(cudaFuncSetAttribute(depthwise_rxr_kernel<2, 5>, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024));
            attr_set[dev] = 1;
        }
    }
    if (smem > 100 * 1024) return CPRUNE_ERR_UNSUPPORTED;
    const int threads = ((p.TW * p.G + 31) / 32) * 32;
    if (i.R == 5) {
        if (i.stride == 1) CPRUNE_CUDA_CHECK(launch_chained(depthwise_rxr_kernel<1, 5>, dim3((unsigned)blocks), dim3(threads), (size_t)smem, st, tm, p));
        else CPRUNE_CUDA_CHECK(launch_chained(depthwise_rxr_kernel<2, 5>, dim3((unsigned)blocks), dim3(threads), (size_t)smem, st, tm, p));
    } else if (i.stride == 1) {
        CPRUNE_CUDA_CHECK(launch_chained(depthwise3x3_kernel<1>, dim3((unsigned)blocks), dim3(threads), (size_t)smem, st, tm, p));
    } else {
        CPRUNE_CUDA_CHECK(launch_chained(depthwise3x3_kernel<2>, dim3((unsigned)blocks), dim3(threads), (size_t)smem, st, tm, p));
    }
    CPRUNE_LAUNCH_CHECK("depthwise kernel");
    return CPRUNE_OK;
}

}  // namespace cprune
