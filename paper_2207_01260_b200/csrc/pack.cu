// Layout changes: filter packing (float32 KCRS -> bf16 KRSC, channel padded), the input cast
// (float32 NHWC -> bf16 NHWC padded) and the widening of bf16 results to float32.
#include "common.cuh"
#include "plan.h"

namespace cprune {

// dense: out[k][r][s'][c] for k < k_alloc, s' < S_out, c < c_pad, where tap s' holds filter tap s = s' - s_off
// (s_off = 1 puts one zero tap in front of every filter row); zero where k >= K, c >= C or s is out of range
__global__ void pack_dense_kernel(const float *__restrict__ w, int K, int C, int R, int S, int S_out, int s_off, int k_alloc,
                                  int c_pad, __nv_bfloat16 *__restrict__ out) {
    size_t total = (size_t)k_alloc * R * S_out * c_pad;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
        int c = (int)(e % c_pad);
        size_t t = e / c_pad;
        int s = (int)(t % S_out) - s_off;
        t /= S_out;
        int r = (int)(t % R);
        int k = (int)(t / R);
        float v = (k < K && c < C && s >= 0 && s < S) ? w[(((size_t)k * C + c) * R + r) * S + s] : 0.f;
        out[e] = __float2bfloat16_rn(v);
    }
}

// depthwise: w [C][1][R][S] -> out[r][s][c], c < c_pad
__global__ void pack_depthwise_kernel(const float *__restrict__ w, int C, int R, int S, int c_pad,
                                      __nv_bfloat16 *__restrict__ out) {
    size_t total = (size_t)R * S * c_pad;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
        int c = (int)(e % c_pad);
        int rs = (int)(e / c_pad);
        float v = c < C ? w[(size_t)c * R * S + rs] : 0.f;
        out[e] = __float2bfloat16_rn(v);
    }
}

__global__ void pad_bias_kernel(const float *__restrict__ b, int K, int k_alloc, float *__restrict__ out) {
    int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k < k_alloc) out[k] = (b && k < K) ? b[k] : 0.f;
}

// one thread per (pixel, group of 8 output lanes)
__global__ void cast_input_kernel(const float *__restrict__ x, size_t pixels, int C, int c_pad, bf16x8 *__restrict__ y) {
    pdl_trigger();
    pdl_wait();
    int groups = c_pad / 8;
    size_t total = pixels * groups;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
        size_t pix = e / groups;
        int g = (int)(e - pix * groups);
        float f[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            int c = g * 8 + i;
            f[i] = c < C ? x[pix * C + c] : 0.f;
        }
        y[e] = pack8(f);
    }
}

__global__ void widen_kernel(const __nv_bfloat16 *__restrict__ x, size_t n, float *__restrict__ y) {
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x)
        y[e] = __bfloat162float(x[e]);
}

static int grid_for(size_t total, int threads) {
    size_t g = (total + threads - 1) / threads;
    if (g < 1) g = 1;
    if (g > 148 * 32) g = 148 * 32;
    return (int)g;
}

cprune_status pack_dense(const float *w, const float *b, int K, int C, int R, int S, int S_out, int k_alloc, int c_pad,
                         void *w_packed, float *b_packed, cudaStream_t st) {
    size_t total = (size_t)k_alloc * R * S_out * c_pad;
    pack_dense_kernel<<<grid_for(total, 256), 256, 0, st>>>(w, K, C, R, S, S_out, S_out - S, k_alloc, c_pad,
                                                           (__nv_bfloat16 *)w_packed);
    CPRUNE_LAUNCH_CHECK("pack_dense_kernel");
    pad_bias_kernel<<<(k_alloc + 255) / 256, 256, 0, st>>>(b, K, k_alloc, b_packed);
    CPRUNE_LAUNCH_CHECK("pad_bias_kernel");
    return CPRUNE_OK;
}

}  // namespace cprune

using namespace cprune;

extern "C" {

cprune_status cprune_pack_weights(const cprune_plan *plan, const float *w, const float *b, void *w_packed,
                                  float *b_packed, void *stream) {
    if (!plan || !w || !w_packed || !b_packed) return CPRUNE_ERR_INVALID_ARG;
    const cprune_plan_info &i = plan->info;
    cudaStream_t st = (cudaStream_t)stream;
    if (i.kernel == CPRUNE_KERNEL_DEPTHWISE) {
        size_t total = (size_t)i.R * i.S * i.c_pad;
        pack_depthwise_kernel<<<grid_for(total, 256), 256, 0, st>>>(w, i.C, i.R, i.S, i.c_pad, (__nv_bfloat16 *)w_packed);
        CPRUNE_LAUNCH_CHECK("pack_depthwise_kernel");
        pad_bias_kernel<<<(i.k_alloc + 255) / 256, 256, 0, st>>>(b, i.K, i.k_alloc, b_packed);
        CPRUNE_LAUNCH_CHECK("pad_bias_kernel");
        return CPRUNE_OK;
    }
    if (i.kernel == CPRUNE_KERNEL_TENSOR && plan->patch && plan->narrow) {
        pad_bias_kernel<<<(i.k_alloc + 255) / 256, 256, 0, st>>>(b, i.K, i.k_alloc, b_packed);
        CPRUNE_LAUNCH_CHECK("pad_bias_kernel");
        return pack_conv_patch(plan, w, w_packed, st);
    }
    const int s_out = (i.kernel == CPRUNE_KERNEL_TENSOR && plan->s_packed > 0) ? plan->s_packed : i.S;
    return pack_dense(w, b, i.K, i.C, i.R, i.S, s_out, i.k_alloc, i.c_pad, w_packed, b_packed, st);
}

cprune_status cprune_fc_pack(const float *w, const float *b, int out, int in, void *w_packed, float *b_packed,
                             void *stream) {
    if (!w || !w_packed || !b_packed || out <= 0 || in <= 0) return CPRUNE_ERR_INVALID_ARG;
    return pack_dense(w, b, out, in, 1, 1, 1, cprune_padded_channels(out), cprune_padded_channels(in), w_packed, b_packed,
                      (cudaStream_t)stream);
}

cprune_status cprune_cast_input(const float *x, size_t pixels, int C, void *y, void *stream) {
    if (!x || !y || C <= 0) return CPRUNE_ERR_INVALID_ARG;
    if (pixels == 0) return CPRUNE_OK;
    int c_pad = cprune_padded_channels(C);
    CPRUNE_CUDA_CHECK(launch_chained(cast_input_kernel, dim3(grid_for(pixels * (c_pad / 8), 256)), dim3(256), 0, (cudaStream_t)stream, x, pixels, C,
                                     c_pad, (bf16x8 *)y));
    return CPRUNE_OK;
}

cprune_status cprune_widen_output(const void *x, size_t count, float *y, void *stream) {
    if (!x || !y) return CPRUNE_ERR_INVALID_ARG;
    if (count == 0) return CPRUNE_OK;
    widen_kernel<<<grid_for(count, 256), 256, 0, (cudaStream_t)stream>>>((const __nv_bfloat16 *)x, count, y);
    CPRUNE_LAUNCH_CHECK("widen_kernel");
    return CPRUNE_OK;
}

}  // extern "C"
