// L1-norm filter selection and slicing (paper Sec. 3.5, last paragraph; Sec. 2.1 / Fig. 2).
//
// Four small kernels, all on the caller's stream:
//   l1_norm_kernel   one CTA per filter: n_k = sum rint(|w| * 2^40) as int64 (order independent)
//   rank_kernel      rank_k = #{j : n_j > n_k or (n_j == n_k and j < k)};  keep_k = rank_k < keep
//   compact_kernel   ascending list of the kept indices (single CTA, chunked block scan)
//   gather kernels   w[kept], b[kept], w_next[:, kept] (or w_next[kept] for a depthwise consumer)
#include <mutex>
#include <string>

#include "common.cuh"

namespace cprune {

__device__ int g_status_word;

static thread_local std::string t_last_error;

cprune_status cuda_fail(cudaError_t e, const char *what) {
    t_last_error = std::string(what) + ": " + cudaGetErrorString(e);
    (void)cudaGetLastError();
    return CPRUNE_ERR_CUDA;
}

int *device_status_word() {
    static std::mutex mu;
    static int *ptrs[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!ptrs[dev]) {
        int *p = nullptr;
        if (cudaGetSymbolAddress((void **)&p, g_status_word) != cudaSuccess) return nullptr;
        ptrs[dev] = p;
    }
    return ptrs[dev];
}

constexpr int NORM_THREADS = 256;

// accumulate != 0: the norm is added to what norms[] holds (integer adds: any order gives the same bits)
__global__ void __launch_bounds__(NORM_THREADS) l1_norm_kernel(const float *__restrict__ w, size_t inner,
                                                                long long *__restrict__ norms, int *status, int accumulate) {
    const float *row = w + (size_t)blockIdx.x * inner;
    long long acc = 0;
    bool bad = false;
    for (size_t i = threadIdx.x; i < inner; i += NORM_THREADS) {
        float a = fabsf(row[i]);
        bad |= !(a < 1024.f);  // also catches NaN and Inf
        acc += __double2ll_rn((double)a * 1099511627776.0);
    }
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    __shared__ long long part[NORM_THREADS / 32];
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
    if (bad) atomicOr(status, STATUS_BAD_DATA);
    __syncthreads();
    if (threadIdx.x == 0) {
        long long s = 0;
        for (int i = 0; i < NORM_THREADS / 32; ++i) s += part[i];
        norms[blockIdx.x] = accumulate ? norms[blockIdx.x] + s : s;
    }
}

constexpr int RANK_THREADS = 256;

__global__ void __launch_bounds__(RANK_THREADS) rank_kernel(const long long *__restrict__ norms, int K, int keep_k,
                                                             int *__restrict__ keep) {
    __shared__ long long tile[RANK_THREADS];
    int k = blockIdx.x * RANK_THREADS + threadIdx.x;
    long long mine = k < K ? norms[k] : 0;
    int rank = 0;
    for (int base = 0; base < K; base += RANK_THREADS) {
        int j = base + threadIdx.x;
        tile[threadIdx.x] = j < K ? norms[j] : 0;
        __syncthreads();
        int lim = min(RANK_THREADS, K - base);
        for (int t = 0; t < lim; ++t) {
            long long other = tile[t];
            int jj = base + t;
            rank += (other > mine) || (other == mine && jj < k);
        }
        __syncthreads();
    }
    if (k < K) keep[k] = rank < keep_k ? 1 : 0;
}

constexpr int COMPACT_THREADS = 1024;

__global__ void __launch_bounds__(COMPACT_THREADS) compact_kernel(const int *__restrict__ keep, int K,
                                                                  int *__restrict__ kept_idx) {
    __shared__ int warp_sum[COMPACT_THREADS / 32];
    __shared__ int running;
    if (threadIdx.x == 0) running = 0;
    __syncthreads();
    for (int base = 0; base < K; base += COMPACT_THREADS) {
        int k = base + threadIdx.x;
        int f = k < K ? keep[k] : 0;
        int incl = f;
        for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(0xffffffffu, incl, o);
            if ((threadIdx.x & 31) >= o) incl += t;
        }
        if ((threadIdx.x & 31) == 31) warp_sum[threadIdx.x >> 5] = incl;
        __syncthreads();
        int before = running;
        for (int wi = 0; wi < (int)(threadIdx.x >> 5); ++wi) before += warp_sum[wi];
        if (f) kept_idx[before + incl - 1] = k;
        __syncthreads();
        if (threadIdx.x == COMPACT_THREADS - 1) running = before + incl;
        __syncthreads();
    }
}

// out[j][i] = in[idx[j]][i]
__global__ void gather_rows_kernel(const float *__restrict__ in, size_t inner, const int *__restrict__ idx,
                                   int n_idx, float *__restrict__ out) {
    size_t total = (size_t)n_idx * inner;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
        size_t j = e / inner, i = e - j * inner;
        out[e] = in[(size_t)idx[j] * inner + i];
    }
}

// out[o][j][i] = in[o][idx[j]][i]
__global__ void gather_cols_kernel(const float *__restrict__ in, int outer, int cols, size_t inner,
                                   const int *__restrict__ idx, int n_idx, float *__restrict__ out) {
    size_t total = (size_t)outer * n_idx * inner;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
        size_t i = e % inner;
        size_t t = e / inner;
        size_t j = t % n_idx, o = t / n_idx;
        out[e] = in[((size_t)o * cols + idx[j]) * inner + i];
    }
}

// Scratch of the allocation-free entry point: norms (int64) followed by keep flags (int32) for up
// to CPRUNE_SELECT_STATIC_MAX_FILTERS filters.  In host code this name is only a handle for
// cudaGetSymbolAddress, never a pointer that a kernel may be given.
constexpr size_t STATIC_NORM_BYTES = (size_t)CPRUNE_SELECT_STATIC_MAX_FILTERS * sizeof(long long);
constexpr size_t STATIC_KEEP_BYTES = (size_t)CPRUNE_SELECT_STATIC_MAX_FILTERS * sizeof(int);
static __device__ __align__(256) unsigned char g_select_scratch[STATIC_NORM_BYTES + STATIC_KEEP_BYTES];

// Device address of g_select_scratch on the current device, looked up once per device.
static cprune_status select_scratch_address(unsigned char **out) {
    static std::mutex mu;
    static unsigned char *ptrs[64] = {nullptr};
    int dev = 0;
    CPRUNE_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return CPRUNE_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(mu);
    if (!ptrs[dev]) {
        unsigned char *p = nullptr;
        CPRUNE_CUDA_CHECK(cudaGetSymbolAddress((void **)&p, g_select_scratch));
        ptrs[dev] = p;
    }
    *out = ptrs[dev];
    return CPRUNE_OK;
}

static int grid_for(size_t total, int threads) {
    size_t g = (total + threads - 1) / threads;
    if (g < 1) g = 1;
    if (g > 148 * 16) g = 148 * 16;
    return (int)g;
}

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

cprune_status select_launch(const float *w, const float *b, int K, int C, int R, int S, int keep_k,
                            const float *w_next, int K2, int R2, int S2, int next_is_depthwise, int32_t *kept_idx,
                            float *w_out, float *b_out, float *w_next_out, long long *norms, int *keep,
                            int *status, cudaStream_t st) {
    size_t inner = (size_t)C * R * S;
    l1_norm_kernel<<<K, NORM_THREADS, 0, st>>>(w, inner, norms, status, 0);
    CPRUNE_LAUNCH_CHECK("l1_norm_kernel");
    rank_kernel<<<(K + RANK_THREADS - 1) / RANK_THREADS, RANK_THREADS, 0, st>>>(norms, K, keep_k, keep);
    CPRUNE_LAUNCH_CHECK("rank_kernel");
    compact_kernel<<<1, COMPACT_THREADS, 0, st>>>(keep, K, kept_idx);
    CPRUNE_LAUNCH_CHECK("compact_kernel");
    gather_rows_kernel<<<grid_for((size_t)keep_k * inner, 256), 256, 0, st>>>(w, inner, kept_idx, keep_k, w_out);
    CPRUNE_LAUNCH_CHECK("gather_rows_kernel");
    if (b) {
        gather_rows_kernel<<<grid_for(keep_k, 256), 256, 0, st>>>(b, 1, kept_idx, keep_k, b_out);
        CPRUNE_LAUNCH_CHECK("gather_rows_kernel");
    }
    if (w_next) {
        size_t in2 = (size_t)R2 * S2;
        if (next_is_depthwise) {
            gather_rows_kernel<<<grid_for((size_t)keep_k * in2, 256), 256, 0, st>>>(w_next, in2, kept_idx, keep_k,
                                                                                    w_next_out);
        } else {
            gather_cols_kernel<<<grid_for((size_t)K2 * keep_k * in2, 256), 256, 0, st>>>(w_next, K2, K, in2, kept_idx,
                                                                                         keep_k, w_next_out);
        }
        CPRUNE_LAUNCH_CHECK("gather consumer");
    }
    return CPRUNE_OK;
}

}  // namespace cprune

using namespace cprune;

extern "C" {

const char *cprune_status_string(cprune_status s) {
    switch (s) {
        case CPRUNE_OK: return "ok";
        case CPRUNE_ERR_INVALID_ARG: return "invalid argument";
        case CPRUNE_ERR_UNSUPPORTED: return "unsupported";
        case CPRUNE_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case CPRUNE_ERR_CUDA: return "CUDA error";
        case CPRUNE_ERR_TIMEOUT: return "device-side wait timed out";
        case CPRUNE_ERR_INTERNAL: return "internal error";
        case CPRUNE_ERR_BAD_DATA: return "non-finite or out-of-range weight";
    }
    return "unknown status";
}

const char *cprune_last_cuda_error(void) { return t_last_error.c_str(); }

int cprune_padded_channels(int C) { return C <= 0 ? 0 : (C <= 128 ? (C + 7) / 8 * 8 : (C + 15) / 16 * 16); }

size_t cprune_select_workspace_bytes(int K) {
    if (K <= 0) return 0;
    return align_up((size_t)K * sizeof(long long), 256) + align_up((size_t)K * sizeof(int), 256);
}

cprune_status cprune_select_filters(const float *w, const float *b, int K, int C, int R, int S, int keep_k,
                                    const float *w_next, int K2, int R2, int S2, int next_is_depthwise,
                                    int32_t *kept_idx, float *w_out, float *b_out, float *w_next_out,
                                    void *workspace, size_t workspace_bytes, void *stream) {
    if (!w || !kept_idx || !w_out || K <= 0 || C <= 0 || R <= 0 || S <= 0) return CPRUNE_ERR_INVALID_ARG;
    if (keep_k < 1 || keep_k > K) return CPRUNE_ERR_INVALID_ARG;
    if (b && !b_out) return CPRUNE_ERR_INVALID_ARG;
    if (w_next && (!w_next_out || R2 <= 0 || S2 <= 0 || (!next_is_depthwise && K2 <= 0))) return CPRUNE_ERR_INVALID_ARG;
    if ((size_t)C * R * S > 8192) return CPRUNE_ERR_UNSUPPORTED;
    if (!workspace || ((uintptr_t)workspace & 15)) return CPRUNE_ERR_INVALID_ARG;
    if (workspace_bytes < cprune_select_workspace_bytes(K)) return CPRUNE_ERR_WORKSPACE_TOO_SMALL;
    int *status = device_status_word();
    if (!status) return cuda_fail(cudaGetLastError(), "status word");
    long long *norms = (long long *)workspace;
    int *keep = (int *)((char *)workspace + align_up((size_t)K * sizeof(long long), 256));
    return select_launch(w, b, K, C, R, S, keep_k, w_next, K2, R2, S2, next_is_depthwise, kept_idx, w_out, b_out,
                         w_next_out, norms, keep, status, (cudaStream_t)stream);
}

cprune_status cprune_select_filters_static(const float *w, const float *b, int K, int C, int R, int S, int keep_k,
                                           const float *w_next, int K2, int R2, int S2, int next_is_depthwise,
                                           int32_t *kept_idx, float *w_out, float *b_out, float *w_next_out,
                                           void *stream) {
    if (!w || !kept_idx || !w_out || K <= 0 || C <= 0 || R <= 0 || S <= 0) return CPRUNE_ERR_INVALID_ARG;
    if (keep_k < 1 || keep_k > K) return CPRUNE_ERR_INVALID_ARG;
    if (b && !b_out) return CPRUNE_ERR_INVALID_ARG;
    if (w_next && (!w_next_out || R2 <= 0 || S2 <= 0 || (!next_is_depthwise && K2 <= 0))) return CPRUNE_ERR_INVALID_ARG;
    if ((size_t)C * R * S > 8192) return CPRUNE_ERR_UNSUPPORTED;
    if (K > CPRUNE_SELECT_STATIC_MAX_FILTERS) return CPRUNE_ERR_WORKSPACE_TOO_SMALL;   // beyond the fixed buffer
    unsigned char *scratch = nullptr;
    cprune_status st = select_scratch_address(&scratch);
    if (st != CPRUNE_OK) return st;
    int *status = device_status_word();
    if (!status) return cuda_fail(cudaGetLastError(), "status word");
    // every norm and keep flag below K is written before it is read, so stale contents are harmless
    long long *norms = (long long *)scratch;
    int *keep = (int *)(scratch + STATIC_NORM_BYTES);
    return select_launch(w, b, K, C, R, S, keep_k, w_next, K2, R2, S2, next_is_depthwise, kept_idx, w_out, b_out,
                         w_next_out, norms, keep, status, (cudaStream_t)stream);
}

cprune_status cprune_select_shared(const float *const *w_list, const size_t *inner, int n_members, int K, int keep_k,
                                   int32_t *kept_idx, void *workspace, size_t workspace_bytes, void *stream) {
    if (!w_list || !inner || n_members < 1 || K <= 0 || !kept_idx) return CPRUNE_ERR_INVALID_ARG;
    if (keep_k < 1 || keep_k > K) return CPRUNE_ERR_INVALID_ARG;
    for (int m = 0; m < n_members; ++m) {
        if (!w_list[m] || inner[m] == 0) return CPRUNE_ERR_INVALID_ARG;
        if (inner[m] > 8192) return CPRUNE_ERR_UNSUPPORTED;
    }
    if ((size_t)n_members > (size_t)1 << 9) return CPRUNE_ERR_UNSUPPORTED;   // keeps the int64 sums far from overflow
    if (!workspace || ((uintptr_t)workspace & 15)) return CPRUNE_ERR_INVALID_ARG;
    if (workspace_bytes < cprune_select_workspace_bytes(K)) return CPRUNE_ERR_WORKSPACE_TOO_SMALL;
    int *status = device_status_word();
    if (!status) return cuda_fail(cudaGetLastError(), "status word");
    cudaStream_t st = (cudaStream_t)stream;
    long long *norms = (long long *)workspace;
    int *keep = (int *)((char *)workspace + align_up((size_t)K * sizeof(long long), 256));
    for (int m = 0; m < n_members; ++m) {
        l1_norm_kernel<<<K, NORM_THREADS, 0, st>>>(w_list[m], inner[m], norms, status, m > 0);
        CPRUNE_LAUNCH_CHECK("l1_norm_kernel");
    }
    rank_kernel<<<(K + RANK_THREADS - 1) / RANK_THREADS, RANK_THREADS, 0, st>>>(norms, K, keep_k, keep);
    CPRUNE_LAUNCH_CHECK("rank_kernel");
    compact_kernel<<<1, COMPACT_THREADS, 0, st>>>(keep, K, kept_idx);
    CPRUNE_LAUNCH_CHECK("compact_kernel");
    return CPRUNE_OK;
}

cprune_status cprune_gather_rows(const float *in, int rows, size_t inner, const int32_t *idx, int n_idx, float *out,
                                 void *stream) {
    if (!in || !idx || !out || rows <= 0 || inner == 0 || n_idx <= 0 || n_idx > rows) return CPRUNE_ERR_INVALID_ARG;
    gather_rows_kernel<<<grid_for((size_t)n_idx * inner, 256), 256, 0, (cudaStream_t)stream>>>(in, inner, idx, n_idx, out);
    CPRUNE_LAUNCH_CHECK("gather_rows_kernel");
    return CPRUNE_OK;
}

cprune_status cprune_gather_columns(const float *in, int outer, int cols, size_t inner, const int32_t *idx, int n_idx,
                                    float *out, void *stream) {
    if (!in || !idx || !out || outer <= 0 || cols <= 0 || inner == 0 || n_idx <= 0 || n_idx > cols)
        return CPRUNE_ERR_INVALID_ARG;
    gather_cols_kernel<<<grid_for((size_t)outer * n_idx * inner, 256), 256, 0, (cudaStream_t)stream>>>(
        in, outer, cols, inner, idx, n_idx, out);
    CPRUNE_LAUNCH_CHECK("gather_cols_kernel");
    return CPRUNE_OK;
}

cprune_status cprune_poll_device_status(void *stream) {
    int *status = device_status_word();
    if (!status) return cuda_fail(cudaGetLastError(), "status word");
    int h = 0;
    cudaStream_t st = (cudaStream_t)stream;
    CPRUNE_CUDA_CHECK(cudaMemcpyAsync(&h, status, sizeof(int), cudaMemcpyDeviceToHost, st));
    CPRUNE_CUDA_CHECK(cudaStreamSynchronize(st));
    if (h) {
        CPRUNE_CUDA_CHECK(cudaMemsetAsync(status, 0, sizeof(int), st));
        CPRUNE_CUDA_CHECK(cudaStreamSynchronize(st));
    }
    if (h & STATUS_TIMEOUT) return CPRUNE_ERR_TIMEOUT;
    if (h & STATUS_BAD_DATA) return CPRUNE_ERR_BAD_DATA;
    return CPRUNE_OK;
}

}  // extern "C"
