// Depthwise 3x3 task (groups == C == K): memory-bound, CUDA cores.  bf16 NHWC in and out with
// padded channels, float32 arithmetic, fused bias + activation (+ residual).  Threads are laid out
// with the channel group fastest, so that a warp reads consecutive 16-byte vectors of one pixel
// and its neighbours; each thread produces TQ adjacent output columns and reuses the input
// columns they share.
#include "common.cuh"
#include "plan.h"

namespace cprune {

struct DwParams {
    const bf16x8 *x;
    const bf16x8 *w;   // [3][3][c8]
    const float *b;
    const bf16x8 *res;
    bf16x8 *y;
    int N, H, W, P, Q, stride, pad, act;
    int c8;
    int qt;            // ceil(Q / TQ)
    long long items;   // N * P * qt * c8
};

template <int TQ, int STRIDE>
__global__ void __launch_bounds__(256) depthwise3x3_kernel(const DwParams p) {
    long long item = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (item >= p.items) return;
    int cg = (int)(item % p.c8);
    long long t = item / p.c8;
    int qb = (int)(t % p.qt) * TQ;
    t /= p.qt;
    int pp = (int)(t % p.P);
    int n = (int)(t / p.P);

    constexpr int COLS = (TQ - 1) * STRIDE + 3;  // input columns feeding TQ outputs
    float acc[TQ][8];
#pragma unroll
    for (int j = 0; j < TQ; ++j)
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[j][i] = 0.f;

    const int v0 = qb * STRIDE - p.pad;
#pragma unroll
    for (int r = 0; r < 3; ++r) {
        int h = pp * STRIDE - p.pad + r;
        if (h < 0 || h >= p.H) continue;
        float wf[3][8];
#pragma unroll
        for (int s = 0; s < 3; ++s) unpack8(ldg8(p.w + (size_t)(r * 3 + s) * p.c8 + cg), wf[s]);
        const bf16x8 *row = p.x + ((size_t)n * p.H + h) * p.W * p.c8 + cg;
#pragma unroll
        for (int col = 0; col < COLS; ++col) {
            int v = v0 + col;
            if (v < 0 || v >= p.W) continue;
            float xf[8];
            unpack8(ldg8(row + (size_t)v * p.c8), xf);
#pragma unroll
            for (int j = 0; j < TQ; ++j) {
                int s = col - j * STRIDE;
                if (s >= 0 && s < 3) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) acc[j][i] = fmaf(xf[i], wf[s][i], acc[j][i]);
                }
            }
        }
    }
    float bf[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) bf[i] = p.b[cg * 8 + i];
#pragma unroll
    for (int j = 0; j < TQ; ++j) {
        int q = qb + j;
        if (q >= p.Q) break;
        size_t o = (((size_t)n * p.P + pp) * p.Q + q) * p.c8 + cg;
        float rf[8];
        if (p.res) unpack8(p.res[o], rf);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float v = acc[j][i] + bf[i];
            if (p.res) v += rf[i];
            acc[j][i] = apply_act(v, p.act);
        }
        p.y[o] = pack8(acc[j]);
    }
}

cprune_status launch_depthwise(const cprune_plan *plan, const void *x, const void *w, const float *b,
                               const void *res, void *y, cudaStream_t st) {
    const cprune_plan_info &i = plan->info;
    DwParams p;
    p.x = (const bf16x8 *)x;
    p.w = (const bf16x8 *)w;
    p.b = b;
    p.res = (const bf16x8 *)res;
    p.y = (bf16x8 *)y;
    p.N = i.N; p.H = i.H; p.W = i.W; p.P = i.P; p.Q = i.Q;
    p.stride = i.stride; p.pad = i.pad; p.act = plan->opts.activation;
    p.c8 = i.c_pad / 8;
    const int TQ = i.tile_n;  // output columns per thread, chosen by the plan
    p.qt = (i.Q + TQ - 1) / TQ;
    p.items = (long long)i.N * i.P * p.qt * p.c8;
    if (p.items == 0) return CPRUNE_OK;
    long long blocks = ceil_div(p.items, 256);
    if (blocks > 0x7fffffffLL) return CPRUNE_ERR_UNSUPPORTED;
    if (i.stride == 1 && TQ == 4) depthwise3x3_kernel<4, 1><<<(unsigned)blocks, 256, 0, st>>>(p);
    else if (i.stride == 1 && TQ == 2) depthwise3x3_kernel<2, 1><<<(unsigned)blocks, 256, 0, st>>>(p);
    else if (i.stride == 1 && TQ == 1) depthwise3x3_kernel<1, 1><<<(unsigned)blocks, 256, 0, st>>>(p);
    else if (i.stride == 2 && TQ == 2) depthwise3x3_kernel<2, 2><<<(unsigned)blocks, 256, 0, st>>>(p);
    else if (i.stride == 2 && TQ == 1) depthwise3x3_kernel<1, 2><<<(unsigned)blocks, 256, 0, st>>>(p);
    else return CPRUNE_ERR_INTERNAL;
    CPRUNE_LAUNCH_CHECK("depthwise3x3_kernel");
    return CPRUNE_OK;
}

}  // namespace cprune
