// Internal definition of a task plan and the launchers of the kernel families.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "cprune.h"

// Tiling of the patch kernel (conv_patch.cu): a tile is TH output rows of one image, MT blocks of 128 accumulator
// rows, FT filters.
struct PatchTiling {
    int MT, TH, FT, tiles_n, tiles_per_img, wstages, resident, acc_bufs, staging_bufs, patch_bytes;
    int TW, tiles_w, step_h, step_w, org;   // tile width, tiles per image row, distance between tiles, origin offset
    int pstages;                            // depth of the patch ring
    int dense;                              // flat tasks: a tile's output is staged as it lies in memory and stored by one bulk copy
    int stage_bytes;                        // shared memory of one staging buffer
    int dense_pitch;                        // dense staging: bytes between neighbouring pixels in the staging buffer
};

struct cprune_plan {
    cprune_plan_info info;
    cprune_task_opts opts;
    int refs;
    // tensor-core family: tensor maps are encoded for a given (x, w) pointer pair and reused
    // while the pointers stay the same
    std::mutex mu;
    const void *map_x = nullptr;
    const void *map_w = nullptr;
    const void *map_y = nullptr;
    const void *map_res = nullptr;
    alignas(64) CUtensorMap tm_a;   // activations (im2col mode)
    alignas(64) CUtensorMap tm_b;   // packed filters
    alignas(64) CUtensorMap tm_y;   // output, for the staged TMA stores
    alignas(64) CUtensorMap tm_res; // residual as an MMA operand (filter-major orientation)
    alignas(64) CUtensorMap tm_id;  // identity matrix
    int smem_bytes = 0;
    int orient = 0;                 // which side of the MMA the pixels are on
    int staging_bufs = 2;
    int fused_pool = 0;             // the 2x2 max-pool runs inside the conv kernel / the split-K finalize kernel
    int splits = 1;                 // split-K slices per output tile
    int ipp = 0;                    // K blocks per slice
    size_t pool_bytes = 0;          // unpooled conv output in the workspace when a 2x2 pool follows
    size_t partial_bytes = 0;       // float32 partial sums in the workspace
    int small_c = 0;                // 3-channel stems: 1 = 8 taps x 8 channels per K block, 2 = pixel pairs
    int s_packed = 0;               // filter taps per row in the packed weights (S, or S + 1 in pair mode)
    int patch = 0;                  // 1: task on the patch kernel (conv_patch.cu)
    int narrow = 0;                 // patch kernel on a regrouped 16-channel input (stems with few channels)
    size_t pre_bytes = 0;           // regrouped input in the workspace
    PatchTiling pt = {};
    double est_us = 0.0;            // the planner's cost-model estimate of the task's time
};

namespace cprune {

// CUDA-core direct convolution, any dense shape (fallback family and small-C stems)
cprune_status launch_conv_direct(const cprune_plan *plan, const void *x, const void *w, const float *b,
                                 const void *res, void *y, cudaStream_t st);
// depthwise 3x3
cprune_status launch_depthwise(cprune_plan *plan, const void *x, const void *w, const float *b,
                               const void *res, void *y, cudaStream_t st);
// channel groups (of 8 channels) one depthwise CTA handles, for c8 groups in the tensor
int depthwise_groups(int c8);
// tcgen05 implicit GEMM
cprune_status plan_conv_tensor(cprune_plan *plan);  // fills tile fields of plan->info; UNSUPPORTED if not eligible
cprune_status launch_conv_tensor(cprune_plan *plan, const void *x, const void *w, const float *b, const void *res,
                                 void *y, void *partial, cudaStream_t st, bool input_regrouped = false);
// stride-1 R x S > 1 tasks with the input patch resident in shared memory (part of the tensor family)
cprune_status plan_conv_patch(cprune_plan *plan);   // UNSUPPORTED if the task is not eligible or would waste the tile
cprune_status launch_conv_patch(cprune_plan *plan, const void *x, const void *w, const float *b, const void *res,
                                void *y, void *scratch, cudaStream_t st, bool input_regrouped = false);
// regrouped 16-channel input of a stem plan (plan->narrow) written to `scratch` from the benchmark's bf16 input or straight
// from the float32 image (cast and regrouping in one pass)
cprune_status regroup_stem_input(const cprune_plan *plan, const void *x, int x_is_f32, void *scratch, cudaStream_t st);
// cprune_task_run with one more option: the regrouped input of a stem plan is already in the workspace
cprune_status task_run_internal(cprune_plan *plan, const void *x, const void *w_packed, const float *b_packed, const void *residual,
                                void *y, void *workspace, cudaStream_t st, bool input_regrouped);
// where in a task's workspace the regrouped stem input lives
inline void *stem_scratch(const cprune_plan *plan, void *workspace) { return (char *)workspace + plan->pool_bytes; }
// filters of a regrouped stem (plan->narrow) and their size
cprune_status pack_conv_patch(const cprune_plan *plan, const float *w, void *w_packed, cudaStream_t st);
size_t packed_weight_bytes_patch(const cprune_plan *plan);
// tiled bf16 tensor map with a 128- or 32-byte swizzle (inner box extent 64 or 16 elements); out-of-bounds
// elements read as zero
cprune_status encode_tiled_bf16_swz(CUtensorMap *map, const void *ptr, int rank, const unsigned long long *dims,
                                    const unsigned long long *strides_bytes, const unsigned *box, int swizzle_bytes, bool for_loads);
// tiled bf16 tensor map without swizzle, out-of-bounds elements read as zero
cprune_status encode_tiled_bf16(CUtensorMap *map, const void *ptr, int rank, const unsigned long long *dims,
                                const unsigned long long *strides_bytes, const unsigned *box);
// adds the float32 partial sums [splits][M][k_alloc] of a split reduction in index order, then bias, residual (bf16 [M][k_pad]
// or NULL) and activation; y bf16 [M][k_pad]
cprune_status launch_splitk_finalize(const float *partial, int splits, long long M, int k_alloc, int k_pad, const float *bias,
                                     const void *res, int act, void *y, cudaStream_t st);
// 2x2 stride-2 max-pool as a separate pass (used when a plan asks for a pool and the conv kernel
// does not fuse it): x [N][H][W][c] -> y [N][H/2][W/2][c]
cprune_status launch_maxpool(const void *x, int N, int H, int W, int c_pad, int k, int stride, int pad, void *y,
                             cudaStream_t st);

}  // namespace cprune
