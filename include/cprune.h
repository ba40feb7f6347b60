/*
 * cprune.h -- C ABI of the B200 (sm_100a) task-execution library for channel-pruned CNNs.
 *
 * The library runs the "tasks" of a pruned network -- fused Conv2d + folded-BatchNorm bias +
 * activation subgraphs (CPrune, arXiv 2207.01260, Sec. 3.1, Sec. 3.4, Sec. 3.5) -- at arbitrary,
 * non-power-of-two channel counts, and performs the L1-norm filter selection and next-layer
 * input-channel slicing that produces those channel counts (Sec. 3.5, last paragraph; Sec. 2.1
 * and Fig. 2 for the tensor roles).
 *
 * Conventions
 *   - Every function returns a cprune_status; none throws, aborts or synchronises the device
 *     unless its comment says so.  Work is enqueued on `stream` (a cudaStream_t passed as void*;
 *     NULL is the default stream).
 *   - "device" pointers are CUDA device pointers owned by the caller; "host" pointers are plain
 *     host memory.  The library owns only the opaque handles it returns.
 *   - Activations in device memory are NHWC bfloat16 with the channel extent padded to
 *     cprune_padded_channels(C): the next multiple of 8 up to 128 channels (every pixel starts
 *     on a 16-byte boundary), the next multiple of 16 above (a 32-byte boundary: bulk tensor
 *     copies whose rows start off a 32-byte boundary were measured at about two thirds of the
 *     speed, which outweighs the extra bytes once they are a few percent); pad lanes must be
 *     zero on input and are written as zero on output.
 *   - Filters in the API are float32 [K][C/groups][R][S] (the paper's c_{i+1} x c_i x k x k).
 *   - The convolution is a cross-correlation, zero padding, dilation 1,
 *     P = floor((H + 2 pad - R) / stride) + 1.
 */
#ifndef CPRUNE_H_
#define CPRUNE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    CPRUNE_OK = 0,
    CPRUNE_ERR_INVALID_ARG = 1,
    CPRUNE_ERR_UNSUPPORTED = 2,
    CPRUNE_ERR_WORKSPACE_TOO_SMALL = 3,
    CPRUNE_ERR_CUDA = 4,      /* a CUDA runtime/driver call failed; see cprune_last_cuda_error() */
    CPRUNE_ERR_TIMEOUT = 5,   /* a bounded device-side wait expired (reported by cprune_poll_device_status) */
    CPRUNE_ERR_INTERNAL = 6,
    CPRUNE_ERR_BAD_DATA = 7   /* a weight was NaN/Inf or too large for the norm grid (reported by poll) */
} cprune_status;

enum { CPRUNE_ACT_NONE = 0, CPRUNE_ACT_RELU = 1, CPRUNE_ACT_RELU6 = 2 };
/* max-pool applied to the activated conv result: 2x2 stride 2 (VGG blocks), or 3x3 stride 2 pad 1 (ResNet stem;
 * padding never wins the maximum) */
enum { CPRUNE_POOL_NONE = 0, CPRUNE_POOL_MAX2X2 = 1, CPRUNE_POOL_MAX3X3S2 = 2 };
/* kernel families a plan can choose */
enum { CPRUNE_KERNEL_AUTO = 0, CPRUNE_KERNEL_DIRECT = 1, CPRUNE_KERNEL_TENSOR = 2, CPRUNE_KERNEL_DEPTHWISE = 3 };
/* option flags of a plan (bits of cprune_task_opts.flags; part of the plan's cache key).  They select between
 * implementations that compute the same values, for tests and measurements:
 *   IM2COL_ONLY             tensor family: never the kernel that keeps the input patch in shared memory
 *   POOL_ON_EPILOGUE_WARPS  fused 3x3 stride-2 pool: pooled by the epilogue warps instead of separate pooling warps */
enum { CPRUNE_FLAG_IM2COL_ONLY = 1, CPRUNE_FLAG_POOL_ON_EPILOGUE_WARPS = 2, CPRUNE_FLAG_ALL = 3 };

typedef struct cprune_plan cprune_plan;
typedef struct cprune_model cprune_model;

const char *cprune_status_string(cprune_status s);
/* Text of the last failing CUDA call on this host thread ("" if none). host pointer, library-owned. */
const char *cprune_last_cuda_error(void);
/* Channel extent in memory of a tensor with C logical channels: the next multiple of 8 (C <= 128) or of 16 (C > 128). */
int cprune_padded_channels(int C);

/* ---------------------------------------------------------------------------------------------
 * Filter selection (paper Sec. 3.5: a filter's importance is the sum of its absolute weights;
 * the filters with the smallest sums are pruned; the next layer loses the matching input
 * channels, Sec. 2.1).
 *
 * The norm of filter k is n_k = sum over (c,r,s) of rint(|w| * 2^40) as a 64-bit integer, so the
 * result does not depend on the order of a parallel reduction and is reproducible bit for bit.
 * The keep_k filters with the largest n_k are kept; among equal norms the lower index is kept.
 *
 *   w          device, float32 [K][C][R][S] (C = input channels per filter)
 *   b          device, float32 [K], or NULL
 *   keep_k     1 <= keep_k <= K
 *   w_next     device, float32, the consumer layer's filters, or NULL:
 *                next_is_depthwise == 0: [K2][K][R2][S2]  -> w_next_out [K2][keep_k][R2][S2]
 *                next_is_depthwise != 0: [K][1][R2][S2]   -> w_next_out [keep_k][1][R2][S2] (K2 ignored)
 *   kept_idx   device, int32 [keep_k], surviving filter indices in ascending order
 *   w_out      device, float32 [keep_k][C][R][S] = w[kept_idx];  b_out [keep_k] (ignored if b NULL)
 *   workspace  device, at least cprune_select_workspace_bytes(K) bytes, 16-byte aligned
 * Preconditions on the data: finite weights with |w| < 2^10 and C*R*S <= 2^13 per filter (so the
 * integer sum cannot overflow); a violation sets CPRUNE_ERR_BAD_DATA in the device status word.
 * Errors: INVALID_ARG for null/shape/keep_k errors, WORKSPACE_TOO_SMALL, CUDA on launch failure.
 * Everything is enqueued on `stream`; nothing is copied to the host.
 */
size_t cprune_select_workspace_bytes(int K);
cprune_status cprune_select_filters(const float *w, const float *b, int K, int C, int R, int S, int keep_k,
                                    const float *w_next, int K2, int R2, int S2, int next_is_depthwise,
                                    int32_t *kept_idx, float *w_out, float *b_out, float *w_next_out,
                                    void *workspace, size_t workspace_bytes, void *stream);

/* The same selection for callers that must not allocate device memory and have no scratch buffer
 * to hand over: code that runs where a cudaMalloc would stall or is forbidden (inside a latency-
 * critical serving loop, under a framework that has already claimed the whole device, in a process
 * whose memory budget is fixed at start-up).  (The paper has no counterpart to this entry point; it
 * exists for the library's users.)  It takes the arguments of cprune_select_filters without the
 * workspace and keeps the per-filter norms and keep flags in a fixed buffer that lives inside the
 * library image: 48 KiB of device memory on every GPU that loads the library, held until the
 * process exits.  The caller still provides every input and output buffer.
 *   - K must not exceed CPRUNE_SELECT_STATIC_MAX_FILTERS; a larger K returns
 *     CPRUNE_ERR_WORKSPACE_TOO_SMALL and launches nothing.
 *   - It calls no allocating routine (no cudaMalloc / cudaFree).  The first call on each device
 *     looks up the buffer's device address once; make that first call outside any stream capture.
 *   - All calls on a device share the one buffer, which keeps whatever the previous call left.
 *     Every entry a call reads it has written first, so nothing needs clearing, but two calls
 *     whose kernels overlap on the GPU (different streams, no ordering between them) race on it:
 *     order them on one stream or with events.
 * Results are bit-identical to cprune_select_filters. */
#define CPRUNE_SELECT_STATIC_MAX_FILTERS 4096
cprune_status cprune_select_filters_static(const float *w, const float *b, int K, int C, int R, int S, int keep_k,
                                           const float *w_next, int K2, int R2, int S2, int next_is_depthwise,
                                           int32_t *kept_idx, float *w_out, float *b_out, float *w_next_out,
                                           void *stream);

/* Dependency-aware selection (paper Sec. 3.5, last paragraph: layers whose outputs meet in a shortcut add
 * lose the same output channels).  The importance of filter index k is the sum, over the n_members layers,
 * of that layer's grid norm of filter k; the keep_k largest are kept, ties keep the lower index.
 *   w_list   HOST array of n_members device pointers, member m is float32 [K][inner[m]]
 *   inner    HOST array: weights per filter of each member (C*R*S), each <= 2^13
 *   kept_idx device, int32 [keep_k], ascending; slice the members and their consumers with the gather calls
 * Workspace as for cprune_select_filters.  With one member the result equals cprune_select_filters'. */
cprune_status cprune_select_shared(const float *const *w_list, const size_t *inner, int n_members, int K, int keep_k,
                                   int32_t *kept_idx, void *workspace, size_t workspace_bytes, void *stream);

/* Row gather out[j][:] = in[idx[j]][:] (inner floats per row) and column gather
 * out[o][j][:] = in[o][idx[j]][:] for further consumers of the same kept_idx (a depthwise layer's
 * bias, the project layer behind a depthwise layer, the first FC layer).  All pointers device. */
cprune_status cprune_gather_rows(const float *in, int rows, size_t inner, const int32_t *idx, int n_idx,
                                 float *out, void *stream);
cprune_status cprune_gather_columns(const float *in, int outer, int cols, size_t inner, const int32_t *idx,
                                    int n_idx, float *out, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Task plans (the analogue of the paper's task table, Sec. 3.1 and Sec. 3.4: subgraphs with the
 * same shape and properties share one task and one program).
 */
typedef struct {
    int activation;   /* CPRUNE_ACT_* */
    int residual;     /* 1: a residual tensor [N][P][Q][k_pad] is added before the activation */
    int pool;         /* CPRUNE_POOL_*: max-pool applied to the activated result */
    int kernel;       /* CPRUNE_KERNEL_AUTO or a forced family (for tests and measurements) */
    int flags;        /* CPRUNE_FLAG_* bits, 0 by default */
} cprune_task_opts;

typedef struct {
    int N, C, H, W, K, R, S, stride, pad, groups;
    int P, Q;                 /* conv output extent */
    int out_h, out_w;         /* stored output extent (after the optional pool) */
    int c_pad, k_pad;         /* channel extents in memory of x and of y */
    int kernel;               /* CPRUNE_KERNEL_* chosen */
    int tile_m, tile_n, tile_k, stages;
    int tiles_m, tiles_n;
    int k_alloc;              /* filter rows in the packed weight tensor (>= k_pad) */
    size_t packed_weight_bytes, packed_bias_bytes, workspace_bytes;
    double flops;             /* 2 N K C P Q R S / groups */
    double algorithmic_bytes; /* bf16 x + bf16 y (+ bf16 residual) + bf16 w + fp32 b, each once */
    double padded_flops;      /* flops the chosen kernel issues, including channel and tile padding */
    int variant;              /* tensor family: 0 = operands gathered per filter tap (im2col loads), 1 = the input patch
                                 of a tile stays in shared memory and every tap reads it (stride-1 tasks, stems),
                                 2 = as 1, for 1x1 tasks whose output tile is one contiguous range of y: staged as it
                                 lies in memory and stored by a single bulk copy */
    int splits;               /* slices of the reduction that go to different CTAs (1: no split); > 1 adds a second launch */
    /* How the program splits the two iterators that run over the filters (paper Sec. 3.5): the compute iterator
     * (filter tiles x instruction-sized groups per tile) and the store iterator (filter tiles x pieces of the memory
     * layout's channel granule per tile: 8 filters up to 128 filters, 16 above, see cprune_padded_channels); each
     * count stands for `unit` filters that one instruction or one store handles and that cannot shrink. */
    int split_compute[2], unit_compute;
    int split_store[2], unit_store;
    double est_us;            /* the planner's own estimate of the task's time (its cost model, microseconds) */
} cprune_plan_info;

/* Host only; launches nothing.  opts == NULL means bias + ReLU, no residual, no pool, AUTO.
 * Plans are cached: an identical (shape, opts) key returns the same handle with its reference
 * count raised.  groups must be 1 or C (depthwise; then K == C and R == S == 3 or 5, stride 1 or 2).
 * The pool option (paper Sec. 3.4: a task is the fused subgraph) is applied to the activated result:
 * CPRUNE_POOL_MAX2X2 needs even P and Q; CPRUNE_POOL_MAX3X3S2 (3x3, stride 2, pad 1) takes any extent.
 * Errors: INVALID_ARG (non-positive extents, output extent < 1, 2x2 pool on odd P/Q), UNSUPPORTED. */
cprune_status cprune_task_plan(int N, int C, int H, int W, int K, int R, int S, int stride, int pad, int groups,
                               const cprune_task_opts *opts, cprune_plan **out);
cprune_status cprune_plan_query(const cprune_plan *plan, cprune_plan_info *out /* host */);
cprune_status cprune_plan_release(cprune_plan *plan);
/* Drops every cached plan that has no outstanding reference; *n_left (host, may be NULL) receives
 * the number of plans still referenced. */
cprune_status cprune_cache_clear(int *n_left);
/* Number of distinct plans in the cache and number of lookups that hit (host, either may be NULL). */
cprune_status cprune_cache_stats(int *n_plans, long long *n_hits);

/* ---------------------------------------------------------------------------------------------
 * Pruning decision (paper Sec. 3.5): how many filters to prune from a task so that the pruned task keeps
 * the structure of its program.  The paper takes, for each of the two iterators over the filters, the
 * smallest slice of its split (product of the factors / largest factor) and prunes the least common
 * multiple of the two.  Here the program is the plan: *step = LCM(unit_compute * prod(split_compute) /
 * max(split_compute), unit_store * prod(split_store) / max(split_store)).  Host only.
 * cprune_task_estimate gives the planner's estimate of the same task with k_new filters (all else equal;
 * it plans that task, which the cache then holds), so that a caller can ask which filter count makes the
 * task a step faster before it prunes anything.  Errors: INVALID_ARG (null, k_new < 1), UNSUPPORTED. */
cprune_status cprune_prune_step(const cprune_plan *plan, int *step /* host */);
cprune_status cprune_task_estimate(const cprune_plan *plan, int k_new, double *est_us /* host */);

/* Task ordering (paper Sec. 3.3): order[0..n) receives the task indices sorted by pruning impact =
 * execution time x number of subgraphs that share the task, largest first; equal impacts keep the lower
 * index first.  Host arrays. */
cprune_status cprune_task_order(const double *times, const int *counts, int n, int *order);

/* One-time layout change of a (pruned) layer's parameters for its plan:
 * w float32 [K][C/groups][R][S] -> bfloat16 (round to nearest even) [k_alloc][R][S][c_pad] with zero
 * padding (depthwise: [R][S][c_pad]; stems that the plan runs on a regrouped input: the plan's own
 * order of taps and channels); b float32 [K] (NULL = zeros) -> float32 [k_alloc] zero padded.
 * The packed layout belongs to the plan: pack with the plan the task will run with.
 * All pointers device; w_packed needs packed_weight_bytes, b_packed packed_bias_bytes. */
cprune_status cprune_pack_weights(const cprune_plan *plan, const float *w, const float *b, void *w_packed,
                                  float *b_packed, void *stream);

/* Runs one task: y = pool(act(conv(x, w) + b + residual)).
 *   x         device, bf16 [N][H][W][c_pad]          residual  device, bf16 [N][P][Q][k_pad] or NULL
 *   y         device, bf16 [N][out_h][out_w][k_pad]  workspace device, workspace_bytes (may be NULL if 0)
 * The workspace holds what the plan needs besides x and y: float32 partial sums of a split reduction,
 * the unpooled result when the pool runs as a separate pass, the regrouped input of a stem.
 * Enqueue only (at most three launches), no allocation, no synchronisation.  Pointers must be 16-byte
 * aligned.  Errors: INVALID_ARG (null pointer, missing workspace, residual mismatch with the plan), CUDA. */
cprune_status cprune_task_run(cprune_plan *plan, const void *x, const void *w_packed, const float *b_packed,
                              const void *residual, void *y, void *workspace, void *stream);

/* float32 [N][H][W][C] -> bf16 [N][H][W][c_pad] (round to nearest even, pad lanes zero). device pointers. */
cprune_status cprune_cast_input(const float *x, size_t pixels, int C, void *y, void *stream);
/* bf16 [n][c_pad] (or any bf16 buffer) -> float32, element-wise widening. device pointers. */
cprune_status cprune_widen_output(const void *x, size_t count, float *y, void *stream);

/* Stand-alone tail operators on bf16 NHWC tensors with padded channels (device pointers):
 * k x k max-pool (padding never wins), global average pool [N][H][W][c] -> [N][c] (float32
 * accumulation), fully connected y[n][o] = act(b[o] + sum_i x[n][i] w[o][i]) with
 * w bf16 [out_pad][in_pad], b float32 [out_pad], y bf16 [N][out_pad] or float32 [N][out] when
 * out_is_f32. */
cprune_status cprune_maxpool(const void *x, int N, int H, int W, int C, int k, int stride, int pad, void *y, void *stream);
cprune_status cprune_global_avgpool(const void *x, int N, int H, int W, int C, void *y, void *stream);
cprune_status cprune_fc_pack(const float *w, const float *b, int out, int in, void *w_packed, float *b_packed, void *stream);
cprune_status cprune_fc(const void *x, int N, int in, const void *w_packed, const float *b_packed, int out, int act,
                        int out_is_f32, void *y, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Fused inverted-residual block (the MobileNetV2 / MnasNet building block of the paper's Sec. 4.1 models): the three
 * tasks 1x1 expand + activation, 3x3 depthwise (stride 1, pad 1) + activation, 1x1 project (+ the block's input as
 * residual, then act_out) run as ONE kernel that keeps the expanded tensor on the SM.  The result equals that of the
 * three tasks run one after the other (bf16 is rounded at the same places).
 *   x  device bf16 [N][H][W][c_in_pad]        y  device bf16 [N][H][W][k_pad]
 * Supported: stride 1, H * W <= 256 and (H + 2) * (W + 2) <= 256 (one image per thread block), C_in <= 192,
 * C_out <= 256 (<= 192 when H * W > 128); anything else returns CPRUNE_ERR_UNSUPPORTED and the caller runs the three
 * tasks separately.  residual != 0 requires C_in == C_out.  Plans are cached and reference-counted like task plans.
 * cprune_block_pack: float32 w_expand [hidden][C_in], w_depthwise [hidden][1][3][3], w_project [C_out][hidden] and the
 * three biases (each may be NULL = zeros) -> one packed bf16 buffer and one packed float32 bias buffer. */
typedef struct cprune_block cprune_block;
typedef struct {
    int N, C_in, H, W, hidden, C_out, act, act_out, residual;
    int c_in_pad, k_pad, hid_alloc, k_alloc;
    size_t packed_weight_bytes, packed_bias_bytes;
    double flops;               /* 2 N H W (C_in hidden + 9 hidden + hidden C_out) */
    double algorithmic_bytes;   /* x + y + parameters, each once */
    double unfused_bytes;       /* the same with the expanded tensor written and read by three separate tasks */
    int splits;                 /* thread blocks per image (each takes a share of the hidden channels); > 1 adds a second launch */
    size_t workspace_bytes;     /* float32 partial sums of the project layer when splits > 1 */
    double est_us;              /* the planner's estimate (microseconds) */
} cprune_block_info;
cprune_status cprune_block_plan(int N, int C_in, int H, int W, int hidden, int C_out, int act, int act_out, int residual,
                                cprune_block **out);
cprune_status cprune_block_query(const cprune_block *block, cprune_block_info *out /* host */);
cprune_status cprune_block_release(cprune_block *block);
cprune_status cprune_block_pack(const cprune_block *block, const float *w_expand, const float *b_expand, const float *w_depthwise,
                                const float *b_depthwise, const float *w_project, const float *b_project, void *w_packed,
                                float *b_packed, void *stream);
/* Enqueue only (at most two launches), no allocation.  Pointers 16-byte aligned; workspace (device, workspace_bytes) may be
 * NULL when the plan needs none. */
cprune_status cprune_block_run(cprune_block *block, const void *x, const void *w_packed, const float *b_packed, void *y, void *workspace,
                               void *stream);

/* ---------------------------------------------------------------------------------------------
 * Whole models: the aggregate of a network's tasks run back to back (paper Sec. 3.1: the model
 * is compiled as the aggregate of its tasks' programs, and its execution time is measured).
 */
enum { CPRUNE_OP_CONV = 1, CPRUNE_OP_MAXPOOL = 2, CPRUNE_OP_GAP = 3, CPRUNE_OP_FC = 4, CPRUNE_OP_BLOCK = 5 };

typedef struct {
    int op;                 /* CPRUNE_OP_* */
    int in, out, res;       /* tensor ids; 0 is the model input (after the cast to bf16); res < 0: none */
    cprune_plan *plan;      /* CONV: the task's plan (borrowed; must outlive the model) */
    const void *w;          /* CONV / FC: packed weights, device, borrowed */
    const float *b;         /* CONV / FC: packed bias, device, borrowed */
    int p0, p1, p2, p3;     /* MAXPOOL: k, stride, pad, -.  FC: in_features, out_features, activation, - */
    cprune_block *block;    /* BLOCK: the fused block's plan (borrowed); w and b are its packed buffers, res is unused
                               (the block's residual is its own input) */
} cprune_task_desc;

/* Builds a model for input float32 [N][H][W][C].  tasks is a host array, copied.  The output of the
 * last task must be an FC layer; it is written as float32 [N][out_features].  The model allocates
 * its own activation buffers on the current device (cudaMalloc) here, never in cprune_model_run. */
cprune_status cprune_model_create(int N, int H, int W, int C, const cprune_task_desc *tasks, int n_tasks,
                                  cprune_model **out);
/* x device float32 [N][H][W][C]; logits device float32 [N][classes].  Enqueues the cast and every
 * task on `stream`.  With use_graph != 0 the launch sequence is captured into a CUDA graph on the first
 * call for a given (x, logits, stream) and replayed afterwards. */
cprune_status cprune_model_run(cprune_model *model, const float *x, float *logits, int use_graph, void *stream);
/* The same through HOST buffers: x_host float32 [N][H][W][C] and logits_host float32 [N][classes]
 * (pinned memory makes the copies asynchronous).  The call enqueues the host-to-device copy on a
 * private copy stream, the captured launch sequence and the device-to-host copy of the logits on
 * `stream`, and returns without waiting; synchronise `stream` before reading logits_host, and keep
 * x_host unchanged until then.  Two device-side input buffers alternate, so the copy of one call
 * overlaps the kernels of the previous one.  The first call allocates those buffers (cudaMalloc). */
cprune_status cprune_model_run_host(cprune_model *model, const float *x_host, float *logits_host, void *stream);
/* Device pointer and element count of tensor `id` of the model (for tests). */
cprune_status cprune_model_tensor(const cprune_model *model, int id, const void **ptr, int *n, int *h, int *w, int *c_pad);
/* Copies tensor `id` (bf16 [n][h][w][c_pad]) into dst (device) on `stream`. */
cprune_status cprune_model_copy_tensor(const cprune_model *model, int id, void *dst, void *stream);
/* Kernel launches one cprune_model_run enqueues. */
int cprune_model_launches(const cprune_model *model);

/* The model's task table (paper Sec. 3.4: which subgraphs share which task): one entry per distinct plan among
 * the model's conv tasks, in order of first appearance.  entries (host) receives at most max_entries entries;
 * *n_entries the number of distinct tasks. */
typedef struct {
    const cprune_plan *plan;   /* the shared task */
    int count;                 /* subgraphs (conv tasks of the model) that use it */
    int first_task;            /* index into the model's task list of the first of them */
} cprune_task_entry;
cprune_status cprune_model_task_table(const cprune_model *model, cprune_task_entry *entries, int max_entries, int *n_entries);
/* Times every entry of the task table on the device: the entry's first subgraph is run `reps` times back to back
 * on the model's own buffers between two CUDA events (after one untimed run); ms (host, one value per table entry)
 * receives the mean milliseconds per run.  Blocks until the measurements are done.  Feed ms and the counts to
 * cprune_task_order to get the paper's pruning priority. */
cprune_status cprune_model_time_tasks(cprune_model *model, int reps, double *ms, void *stream);
cprune_status cprune_model_destroy(cprune_model *model);

/* Reads and clears the device status word after synchronising `stream` (this call blocks).
 * Returns CPRUNE_OK, CPRUNE_ERR_TIMEOUT or CPRUNE_ERR_BAD_DATA. */
cprune_status cprune_poll_device_status(void *stream);
/* Self-test of the bounded waits: launches one small CTA that waits, with a limit of 65,536 cycles, on a
 * barrier that nothing will ever signal (the same wait routine the tensor-core kernels use with their one-second
 * limit).  The wait gives up, raises the time-out bit of the device status word and the kernel returns; the next
 * cprune_poll_device_status therefore reports CPRUNE_ERR_TIMEOUT once, and the device stays usable. */
cprune_status cprune_selftest_wait_timeout(void *stream);

#ifdef __cplusplus
}
#endif
#endif /* CPRUNE_H_ */
