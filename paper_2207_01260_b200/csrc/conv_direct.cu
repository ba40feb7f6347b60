// CUDA-core convolution kernels: the direct dense kernel (any shape; the fallback family, also
// used for 3-channel stems) and the depthwise 3x3 kernel.  Both read bf16 NHWC with padded
// channels, accumulate in float32 and fuse bias + residual + activation (paper Sec. 3.4: a task is
// Conv2d + BatchNorm (folded) + ReLU).
#include "common.cuh"
#include "plan.h"

namespace cprune {

struct DirectParams {
    const bf16x8 *x;
    const bf16x8 *w;
    const float *b;
    const bf16x8 *res;
    bf16x8 *y;
    int N, H, W, P, Q, R, S, stride, pad, act;
    int c8;        // c_pad / 8
    int k8;        // k_pad / 8
    long long M;   // N * P * Q
};

// one thread: one output pixel, 8 consecutive filters
__global__ void __launch_bounds__(128) conv_direct_kernel(const DirectParams p) {
    long long item = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (item >= p.M * p.k8) return;
    int kg = (int)(item / p.M);
    long long m = item - (long long)kg * p.M;
    int q = (int)(m % p.Q);
    long long t = m / p.Q;
    int pp = (int)(t % p.P);
    int n = (int)(t / p.P);
    float acc[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] = 0.f;
    const size_t wrow = (size_t)p.R * p.S * p.c8;  // 16-byte vectors per filter
    for (int r = 0; r < p.R; ++r) {
        int h = pp * p.stride - p.pad + r;
        if (h < 0 || h >= p.H) continue;
        for (int s = 0; s < p.S; ++s) {
            int v = q * p.stride - p.pad + s;
            if (v < 0 || v >= p.W) continue;
            const bf16x8 *xp = p.x + (((size_t)n * p.H + h) * p.W + v) * p.c8;
            const bf16x8 *wp = p.w + (size_t)kg * 8 * wrow + (size_t)(r * p.S + s) * p.c8;
            for (int c = 0; c < p.c8; ++c) {
                float xf[8];
                unpack8(xp[c], xf);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    float wf[8];
                    unpack8(ldg8(wp + (size_t)j * wrow + c), wf);
#pragma unroll
                    for (int i = 0; i < 8; ++i) acc[j] = fmaf(xf[i], wf[i], acc[j]);
                }
            }
        }
    }
    size_t o = (size_t)m * p.k8 + kg;
    float rf[8];
    if (p.res) unpack8(p.res[o], rf);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        float v = acc[j] + p.b[kg * 8 + j];
        if (p.res) v += rf[j];
        acc[j] = apply_act(v, p.act);
    }
    p.y[o] = pack8(acc);
}

cprune_status launch_conv_direct(const cprune_plan *plan, const void *x, const void *w, const float *b,
                                 const void *res, void *y, cudaStream_t st) {
    const cprune_plan_info &i = plan->info;
    DirectParams p;
    p.x = (const bf16x8 *)x;
    p.w = (const bf16x8 *)w;
    p.b = b;
    p.res = (const bf16x8 *)res;
    p.y = (bf16x8 *)y;
    p.N = i.N; p.H = i.H; p.W = i.W; p.P = i.P; p.Q = i.Q; p.R = i.R; p.S = i.S;
    p.stride = i.stride; p.pad = i.pad; p.act = plan->opts.activation;
    p.c8 = i.c_pad / 8;
    p.k8 = i.k_pad / 8;
    p.M = (long long)i.N * i.P * i.Q;
    long long items = p.M * p.k8;
    if (items == 0) return CPRUNE_OK;
    long long blocks = ceil_div(items, 128);
    if (blocks > 0x7fffffffLL) return CPRUNE_ERR_UNSUPPORTED;
    conv_direct_kernel<<<(unsigned)blocks, 128, 0, st>>>(p);
    CPRUNE_LAUNCH_CHECK("conv_direct_kernel");
    return CPRUNE_OK;
}

}  // namespace cprune
