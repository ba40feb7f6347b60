// Shared host/device helpers of the cprune library (status word, error capture, bf16 vectors).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "cprune.h"

namespace cprune {

// bits of the device status word
enum : int { STATUS_TIMEOUT = 1, STATUS_BAD_DATA = 2 };

// Device address of the per-device status word (resolved once per device).
int *device_status_word();

// Records a failing CUDA call for cprune_last_cuda_error() and returns CPRUNE_ERR_CUDA.
cprune_status cuda_fail(cudaError_t e, const char *what);

#define CPRUNE_CUDA_CHECK(expr)                                     \
    do {                                                            \
        cudaError_t e__ = (expr);                                   \
        if (e__ != cudaSuccess) return ::cprune::cuda_fail(e__, #expr); \
    } while (0)

#define CPRUNE_LAUNCH_CHECK(name)                                   \
    do {                                                            \
        cudaError_t e__ = cudaGetLastError();                       \
        if (e__ != cudaSuccess) return ::cprune::cuda_fail(e__, name); \
    } while (0)

// Programmatic dependent launch.  A kernel of a model's launch chain lets its successor start as early as possible
// (pdl_trigger) and waits for its predecessor's results (pdl_wait) only after its own set-up, so that launch
// latency and set-up overlap the predecessor's tail.  Both are no-ops in a kernel launched the ordinary way.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// True while the calling thread enqueues a chain whose kernels may overlap their predecessors' tails.
bool chain_launch_enabled();
void set_chain_launch(bool on);

// Launches a kernel that calls pdl_wait() before it touches global memory; inside a chain the launch carries the
// programmatic-serialization attribute.
template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    if (chain_launch_enabled()) {
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
    }
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

inline int round_up(int v, int m) { return (v + m - 1) / m * m; }
inline long long ceil_div(long long a, long long b) { return (a + b - 1) / b; }

__device__ __forceinline__ float apply_act(float v, int act) {
    if (act == CPRUNE_ACT_RELU) return fmaxf(v, 0.f);
    if (act == CPRUNE_ACT_RELU6) return fminf(fmaxf(v, 0.f), 6.f);
    return v;
}

// 8 bf16 values carried in one 16-byte vector.  The members are plain words so that a copy of the struct is ONE 16-byte
// load or store (with __nv_bfloat162 members, whose assignment is user-defined, it is four 4-byte ones).
struct alignas(16) bf16x8 {
    uint32_t w[4];
};

__device__ __forceinline__ bf16x8 ldg8(const bf16x8 *p) {
    uint4 u = __ldg(reinterpret_cast<const uint4 *>(p));
    bf16x8 r;
    r.w[0] = u.x; r.w[1] = u.y; r.w[2] = u.z; r.w[3] = u.w;
    return r;
}

__device__ __forceinline__ void unpack8(const bf16x8 &a, float *f) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        // a bf16 is the upper half of the float32 with the same value
        f[2 * i] = __uint_as_float(a.w[i] << 16);
        f[2 * i + 1] = __uint_as_float(a.w[i] & 0xffff0000u);
    }
}

__device__ __forceinline__ bf16x8 pack8(const float *f) {
    bf16x8 r;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __nv_bfloat162 t = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
        r.w[i] = *reinterpret_cast<const uint32_t *>(&t);
    }
    return r;
}

}  // namespace cprune
