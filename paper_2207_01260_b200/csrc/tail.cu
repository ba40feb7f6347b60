// Model-tail operators on bf16 NHWC tensors with padded channels: k x k max-pool, global
// average pool and fully-connected layers.  All are memory-bound; float32 arithmetic.
#include "common.cuh"
#include "plan.h"

namespace cprune {

__global__ void __launch_bounds__(256) maxpool_kernel(const bf16x8 *__restrict__ x, int N, int H, int W, int c8,
                                                      int P, int Q, int k, int stride, int pad,
                                                      bf16x8 *__restrict__ y) {
    pdl_trigger();
    pdl_wait();
    long long total = (long long)N * P * Q * c8;
    long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= total) return;
    int cg = (int)(e % c8);
    long long t = e / c8;
    int q = (int)(t % Q);
    t /= Q;
    int p = (int)(t % P);
    int n = (int)(t / P);
    float m[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) m[i] = -INFINITY;
    for (int r = 0; r < k; ++r) {
        int h = p * stride - pad + r;
        if (h < 0 || h >= H) continue;
        for (int s = 0; s < k; ++s) {
            int v = q * stride - pad + s;
            if (v < 0 || v >= W) continue;
            float f[8];
            unpack8(ldg8(x + (((size_t)n * H + h) * W + v) * c8 + cg), f);
#pragma unroll
            for (int i = 0; i < 8; ++i) m[i] = fmaxf(m[i], f[i]);
        }
    }
    y[e] = pack8(m);
}

// One block per (image, 32 channel groups): 8 pixel lanes x 32 channel groups; each thread sums every 8th pixel of
// its channel group in float32, the lanes are added through shared memory in a fixed order, mean stored as bf16.
__global__ void __launch_bounds__(256) gap_kernel(const bf16x8 *__restrict__ x, int N, int HW, int c8,
                                                  bf16x8 *__restrict__ y) {
    __shared__ float part[8][32][9];
    pdl_trigger();
    pdl_wait();
    const int blocks_per_img = (c8 + 31) / 32;
    const int n = blockIdx.x / blocks_per_img;
    const int cg = (blockIdx.x - n * blocks_per_img) * 32 + (threadIdx.x & 31);
    const int pl = threadIdx.x >> 5;
    float s[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) s[i] = 0.f;
    if (cg < c8) {
        const bf16x8 *px = x + (size_t)n * HW * c8 + cg;
        for (int i = pl; i < HW; i += 8) {
            float f[8];
            unpack8(ldg8(px + (size_t)i * c8), f);
#pragma unroll
            for (int j = 0; j < 8; ++j) s[j] += f[j];
        }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) part[pl][threadIdx.x & 31][j] = s[j];
    __syncthreads();
    if (pl == 0 && cg < c8) {
        float t[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) t[j] = 0.f;
        for (int l = 0; l < 8; ++l)
#pragma unroll
            for (int j = 0; j < 8; ++j) t[j] += part[l][threadIdx.x & 31][j];
        const float inv = 1.f / (float)HW;
#pragma unroll
        for (int j = 0; j < 8; ++j) t[j] *= inv;
        y[(size_t)n * c8 + cg] = pack8(t);
    }
}

// One warp per (OB consecutive output features, group of NB images): the lanes split the input features; every
// activation chunk is used for OB outputs and every weight chunk for NB images, reduced with shuffles at the end.
template <int NB, int OB>
__global__ void __launch_bounds__(256) fc_kernel(const bf16x8 *__restrict__ x, int N, int in8,
                                                 const bf16x8 *__restrict__ w, const float *__restrict__ b, int out,
                                                 int out_pad, int act, int out_is_f32, void *__restrict__ y) {
    pdl_trigger();
    pdl_wait();
    const int ngroups = (N + NB - 1) / NB;
    const long long widx = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (widx >= (long long)(out_pad / OB) * ngroups) return;
    const int o0 = (int)(widx / ngroups) * OB;
    const int n0 = (int)(widx % ngroups) * NB;
    float acc[OB][NB];
#pragma unroll
    for (int q = 0; q < OB; ++q)
#pragma unroll
        for (int j = 0; j < NB; ++j) acc[q][j] = 0.f;
    for (int i = lane; i < in8; i += 32) {
        float wf[OB][8];
#pragma unroll
        for (int q = 0; q < OB; ++q) unpack8(ldg8(w + (size_t)(o0 + q) * in8 + i), wf[q]);
#pragma unroll
        for (int j = 0; j < NB; ++j) {
            if (n0 + j < N) {
                float xf[8];
                unpack8(ldg8(x + (size_t)(n0 + j) * in8 + i), xf);
#pragma unroll
                for (int q = 0; q < OB; ++q)
#pragma unroll
                    for (int t = 0; t < 8; ++t) acc[q][j] = fmaf(xf[t], wf[q][t], acc[q][j]);
            }
        }
    }
    // OB * NB = 32 partial sums per lane -> lane l ends up with the total of sum number l: at every halving step a lane
    // keeps the half of the sums selected by one bit of its index and hands the other half to its partner (31 shuffles
    // instead of 160)
    static_assert(OB * NB == 32, "one total per lane");
    float v[32];
#pragma unroll
    for (int q = 0; q < OB; ++q)
#pragma unroll
        for (int j = 0; j < NB; ++j) v[q * NB + j] = acc[q][j];
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) {
        const bool up = (lane & s) != 0;
#pragma unroll
        for (int i = 0; i < s; ++i) {
            const float keep = up ? v[i + s] : v[i];
            const float give = up ? v[i] : v[i + s];
            v[i] = keep + __shfl_xor_sync(0xffffffffu, give, s);
        }
    }
    {
        const int o = o0 + lane / NB, n = n0 + lane % NB;
        if (n < N) {
            const float r = apply_act(v[0] + b[o], act);
            if (out_is_f32) {
                if (o < out) ((float *)y)[(size_t)n * out + o] = r;
            } else {
                ((__nv_bfloat16 *)y)[(size_t)n * out_pad + o] = __float2bfloat16_rn(o < out ? r : 0.f);
            }
        }
    }
}

cprune_status launch_maxpool(const void *x, int N, int H, int W, int c_pad, int k, int stride, int pad, void *y,
                             cudaStream_t st) {
    int P = (H + 2 * pad - k) / stride + 1, Q = (W + 2 * pad - k) / stride + 1;
    long long total = (long long)N * P * Q * (c_pad / 8);
    if (total == 0) return CPRUNE_OK;
    long long blocks = ceil_div(total, 256);
    if (blocks > 0x7fffffffLL) return CPRUNE_ERR_UNSUPPORTED;
    CPRUNE_CUDA_CHECK(launch_chained(maxpool_kernel, dim3((unsigned)blocks), dim3(256), 0, st, (const bf16x8 *)x, N, H, W, c_pad / 8, P, Q, k,
                                     stride, pad, (bf16x8 *)y));
    return CPRUNE_OK;
}

}  // namespace cprune

using namespace cprune;

extern "C" {

cprune_status cprune_maxpool(const void *x, int N, int H, int W, int C, int k, int stride, int pad, void *y,
                             void *stream) {
    if (!x || !y || N <= 0 || H <= 0 || W <= 0 || C <= 0 || k <= 0 || stride <= 0 || pad < 0 || 2 * pad > k)
        return CPRUNE_ERR_INVALID_ARG;
    if (H + 2 * pad < k || W + 2 * pad < k) return CPRUNE_ERR_INVALID_ARG;
    return launch_maxpool(x, N, H, W, cprune_padded_channels(C), k, stride, pad, y, (cudaStream_t)stream);
}

cprune_status cprune_global_avgpool(const void *x, int N, int H, int W, int C, void *y, void *stream) {
    if (!x || !y || N <= 0 || H <= 0 || W <= 0 || C <= 0) return CPRUNE_ERR_INVALID_ARG;
    int c8 = cprune_padded_channels(C) / 8;
    CPRUNE_CUDA_CHECK(launch_chained(gap_kernel, dim3(N * ((c8 + 31) / 32)), dim3(256), 0, (cudaStream_t)stream, (const bf16x8 *)x, N, H * W, c8,
                                     (bf16x8 *)y));
    return CPRUNE_OK;
}

cprune_status cprune_fc(const void *x, int N, int in, const void *w_packed, const float *b_packed, int out, int act,
                        int out_is_f32, void *y, void *stream) {
    if (!x || !w_packed || !b_packed || !y || N <= 0 || in <= 0 || out <= 0) return CPRUNE_ERR_INVALID_ARG;
    int in8 = cprune_padded_channels(in) / 8, out_pad = cprune_padded_channels(out);
    const int warps = 8;
    const long long total_warps = (long long)(out_pad / 4) * ((N + 7) / 8);
    CPRUNE_CUDA_CHECK(launch_chained(fc_kernel<8, 4>, dim3((unsigned)((total_warps + warps - 1) / warps)), dim3(warps * 32), 0, (cudaStream_t)stream,
                                     (const bf16x8 *)x, N, in8, (const bf16x8 *)w_packed, b_packed, out, out_pad, act, out_is_f32, y));
    return CPRUNE_OK;
}

}  // extern "C"
