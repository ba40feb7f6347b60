// Task plans and the plan cache (paper Sec. 3.1 / Sec. 3.4: subgraphs with identical shape and
// properties map to one task, and each task keeps one program).  A plan is a pure function of its
// key (shape + fused-epilogue options); planning launches nothing and needs no device.
#include <array>
#include <cstdlib>
#include <map>
#include <mutex>

#include "common.cuh"
#include "plan.h"

namespace cprune {

static thread_local bool g_chain_launch = false;
bool chain_launch_enabled() { return g_chain_launch; }
void set_chain_launch(bool on) { g_chain_launch = on; }

using PlanKey = std::array<int, 15>;

struct PlanCache {
    std::mutex mu;
    std::map<PlanKey, cprune_plan *> plans;
    long long hits = 0;
};

static PlanCache &cache() {
    static PlanCache c;
    return c;
}

static cprune_status build_plan(const PlanKey &key, cprune_plan **out) {
    cprune_plan *pl = new cprune_plan();
    cprune_plan_info &i = pl->info;
    i = cprune_plan_info();
    i.N = key[0]; i.C = key[1]; i.H = key[2]; i.W = key[3]; i.K = key[4]; i.R = key[5]; i.S = key[6];
    i.stride = key[7]; i.pad = key[8]; i.groups = key[9];
    pl->opts.activation = key[10]; pl->opts.residual = key[11]; pl->opts.pool = key[12]; pl->opts.kernel = key[13];
    pl->opts.flags = key[14];
    pl->refs = 0;
    i.P = (i.H + 2 * i.pad - i.R) / i.stride + 1;
    i.Q = (i.W + 2 * i.pad - i.S) / i.stride + 1;
    i.out_h = i.P; i.out_w = i.Q;
    if (pl->opts.pool == CPRUNE_POOL_MAX2X2) { i.out_h = i.P / 2; i.out_w = i.Q / 2; }
    if (pl->opts.pool == CPRUNE_POOL_MAX3X3S2) { i.out_h = (i.P - 1) / 2 + 1; i.out_w = (i.Q - 1) / 2 + 1; }
    i.c_pad = cprune_padded_channels(i.C);
    i.k_pad = cprune_padded_channels(i.K);
    i.k_alloc = i.k_pad;
    i.flops = 2.0 * i.N * (double)i.K * (i.C / i.groups) * i.P * i.Q * i.R * i.S;
    i.padded_flops = 2.0 * i.N * (double)i.k_pad * (i.groups == 1 ? i.c_pad : 1) * i.P * i.Q * i.R * i.S;
    const bool depthwise = i.groups > 1;
    int family = pl->opts.kernel;
    cprune_status st = CPRUNE_OK;
    if (depthwise) {
        if (family != CPRUNE_KERNEL_AUTO && family != CPRUNE_KERNEL_DEPTHWISE) st = CPRUNE_ERR_UNSUPPORTED;
        family = CPRUNE_KERNEL_DEPTHWISE;
        // output pixels per CTA (rows x columns) are chosen at launch, see depthwise.cu
        i.tile_m = i.stride == 1 ? 14 : 4;
        i.tile_n = 14;
        i.tile_k = 8;
    } else {
        if (family == CPRUNE_KERNEL_DEPTHWISE) st = CPRUNE_ERR_UNSUPPORTED;
        // 3-channel stems run on the tensor cores too when their filters fit the 128-row side
        if (family == CPRUNE_KERNEL_AUTO) family = (i.C < 8 && i.K > 128) ? CPRUNE_KERNEL_DIRECT : CPRUNE_KERNEL_TENSOR;
        if (st == CPRUNE_OK && family == CPRUNE_KERNEL_TENSOR) {
            cprune_status t = plan_conv_tensor(pl);
            if (t != CPRUNE_OK) {
                if (pl->opts.kernel == CPRUNE_KERNEL_TENSOR) st = t;
                family = CPRUNE_KERNEL_DIRECT;
            }
        }
        if (family == CPRUNE_KERNEL_DIRECT) {
            i.tile_m = 1; i.tile_n = 8; i.tile_k = 8; i.stages = 0;
            i.tiles_m = i.N * i.P * i.Q; i.tiles_n = i.k_pad / 8;
        }
    }
    if (st != CPRUNE_OK) { delete pl; return st; }
    i.kernel = family;
    const double rs = (double)i.R * i.S;
    i.algorithmic_bytes = 2.0 * ((double)i.N * i.H * i.W * i.C + (double)i.N * i.out_h * i.out_w * i.K +
                                 (pl->opts.residual ? (double)i.N * i.P * i.Q * i.K : 0.0) +
                                 (double)i.K * (i.C / i.groups) * rs) + 4.0 * i.K;
    // how the program splits the filter axis (see cprune_prune_step)
    i.splits = family == CPRUNE_KERNEL_TENSOR ? pl->splits : 1;
    if (family == CPRUNE_KERNEL_TENSOR && (pl->patch || pl->orient == 0)) {
        // filters on the MMA's column side: tiles_n tiles of tile_n filters, built from 16-filter instruction groups
        // (64-filter groups when there are several tiles: tiles end on store-box boundaries), stored in pieces of the
        // memory layout's granule (8 filters = 16 bytes up to 128 filters, 16 filters above)
        i.unit_compute = i.tiles_n > 1 ? 64 : 16;
        i.split_compute[0] = i.tiles_n; i.split_compute[1] = i.tile_n / i.unit_compute;
        i.unit_store = i.K > 128 ? 16 : 8;
        i.split_store[0] = i.tiles_n; i.split_store[1] = i.tile_n / i.unit_store;
    } else if (family == CPRUNE_KERNEL_DEPTHWISE) {
        // channel blocks (CTAs along the channels) x channel groups of 8 per CTA
        const int c8 = i.c_pad / 8;
        const int g = depthwise_groups(c8);
        i.unit_compute = i.unit_store = 8;
        i.split_compute[0] = i.split_store[0] = (c8 + g - 1) / g;
        i.split_compute[1] = i.split_store[1] = g;
        pl->est_us = i.algorithmic_bytes / 3.0e6 + 4.0;
    } else {
        // filters on the 128-row side of the MMA (any count up to 128 costs the same) or one thread per 8 filters:
        // the filter axis is only cut into the pieces of the memory layout (8 filters up to 128 filters, 16 above)
        i.unit_compute = i.unit_store = i.K > 128 ? 16 : 8;
        i.split_compute[0] = i.split_store[0] = 1;
        i.split_compute[1] = i.split_store[1] = i.k_pad / i.unit_store;
        if (family == CPRUNE_KERNEL_DIRECT) pl->est_us = i.flops / 15.0e6 + 4.0;
    }
    i.variant = (family == CPRUNE_KERNEL_TENSOR && pl->patch) ? (pl->pt.dense ? 2 : 1) : 0;
    const int s_packed = (family == CPRUNE_KERNEL_TENSOR && pl->s_packed > 0) ? pl->s_packed : i.S;
    i.packed_weight_bytes = depthwise ? (size_t)(rs * i.c_pad * 2) : (size_t)i.k_alloc * i.R * s_packed * i.c_pad * 2;
    if (family == CPRUNE_KERNEL_TENSOR && pl->patch && pl->narrow) i.packed_weight_bytes = packed_weight_bytes_patch(pl);
    i.packed_bias_bytes = (size_t)i.k_alloc * sizeof(float);
    // workspace: [unpooled conv output if a pool follows][split-K partial sums]
    const bool separate_pool = pl->opts.pool != CPRUNE_POOL_NONE && !(family == CPRUNE_KERNEL_TENSOR && pl->fused_pool);
    pl->pool_bytes = separate_pool ? ((size_t)i.N * i.P * i.Q * i.k_pad * 2 + 255) / 256 * 256 : 0;
    // (patch kernel on a regrouped stem: the regrouped input takes the place of the partial sums)
    i.workspace_bytes = pl->pool_bytes + (family == CPRUNE_KERNEL_TENSOR ? pl->partial_bytes + pl->pre_bytes : 0);
    i.est_us = pl->est_us;
    *out = pl;
    return CPRUNE_OK;
}


cprune_status task_run_internal(cprune_plan *plan, const void *x, const void *w_packed, const float *b_packed, const void *residual,
                                void *y, void *workspace, cudaStream_t st, bool input_regrouped) {
    if (!plan || !x || !w_packed || !b_packed || !y) return CPRUNE_ERR_INVALID_ARG;
    if ((plan->opts.residual != 0) != (residual != nullptr)) return CPRUNE_ERR_INVALID_ARG;
    if (((uintptr_t)x | (uintptr_t)w_packed | (uintptr_t)y | (uintptr_t)residual | (uintptr_t)workspace) & 15)
        return CPRUNE_ERR_INVALID_ARG;
    const cprune_plan_info &i = plan->info;
    const bool pool = plan->opts.pool != CPRUNE_POOL_NONE && !(i.kernel == CPRUNE_KERNEL_TENSOR && plan->fused_pool);
    if (i.workspace_bytes && !workspace) return CPRUNE_ERR_INVALID_ARG;
    void *conv_out = pool ? workspace : y;
    void *partial = (plan->partial_bytes || plan->pre_bytes) ? (void *)((char *)workspace + plan->pool_bytes) : nullptr;
    cprune_status s;
    switch (i.kernel) {
        case CPRUNE_KERNEL_TENSOR: s = launch_conv_tensor(plan, x, w_packed, b_packed, residual, conv_out, partial, st, input_regrouped); break;
        case CPRUNE_KERNEL_DIRECT: s = launch_conv_direct(plan, x, w_packed, b_packed, residual, conv_out, st); break;
        case CPRUNE_KERNEL_DEPTHWISE: s = launch_depthwise(plan, x, w_packed, b_packed, residual, conv_out, st); break;
        default: return CPRUNE_ERR_INTERNAL;
    }
    if (s != CPRUNE_OK) return s;
    if (pool) {
        if (plan->opts.pool == CPRUNE_POOL_MAX3X3S2) return launch_maxpool(conv_out, i.N, i.P, i.Q, i.k_pad, 3, 2, 1, y, st);
        return launch_maxpool(conv_out, i.N, i.P, i.Q, i.k_pad, 2, 2, 0, y, st);
    }
    return CPRUNE_OK;
}

}  // namespace cprune

using namespace cprune;

extern "C" {

cprune_status cprune_task_plan(int N, int C, int H, int W, int K, int R, int S, int stride, int pad, int groups,
                               const cprune_task_opts *opts, cprune_plan **out) {
    if (!out) return CPRUNE_ERR_INVALID_ARG;
    *out = nullptr;
    if (N <= 0 || C <= 0 || H <= 0 || W <= 0 || K <= 0 || R <= 0 || S <= 0 || stride <= 0 || pad < 0 || groups <= 0)
        return CPRUNE_ERR_INVALID_ARG;
    if (H + 2 * pad < R || W + 2 * pad < S) return CPRUNE_ERR_INVALID_ARG;
    cprune_task_opts o = {CPRUNE_ACT_RELU, 0, CPRUNE_POOL_NONE, CPRUNE_KERNEL_AUTO, 0};
    if (opts) o = *opts;
    if (o.activation < 0 || o.activation > 2 || o.pool < 0 || o.pool > 2 || o.kernel < 0 || o.kernel > 3 ||
        (o.residual != 0 && o.residual != 1) || (o.flags & ~CPRUNE_FLAG_ALL))
        return CPRUNE_ERR_INVALID_ARG;
    if (groups != 1) {
        if (groups != C || K != C) return CPRUNE_ERR_UNSUPPORTED;
        if (R != S || (R != 3 && R != 5) || stride > 2) return CPRUNE_ERR_UNSUPPORTED;
    }
    int P = (H + 2 * pad - R) / stride + 1, Q = (W + 2 * pad - S) / stride + 1;
    if (o.pool == CPRUNE_POOL_MAX2X2 && ((P & 1) || (Q & 1))) return CPRUNE_ERR_INVALID_ARG;
    if ((long long)N * P * Q > 0x7fffffffLL || (long long)N * H * W > 0x7fffffffLL) return CPRUNE_ERR_UNSUPPORTED;
    PlanKey key = {N, C, H, W, K, R, S, stride, pad, groups, o.activation, o.residual, o.pool, o.kernel, o.flags};
    PlanCache &c = cache();
    std::lock_guard<std::mutex> lock(c.mu);
    auto it = c.plans.find(key);
    if (it != c.plans.end()) {
        ++c.hits;
        ++it->second->refs;
        *out = it->second;
        return CPRUNE_OK;
    }
    cprune_plan *pl = nullptr;
    cprune_status st = build_plan(key, &pl);
    if (st != CPRUNE_OK) return st;
    pl->refs = 1;
    c.plans[key] = pl;
    *out = pl;
    return CPRUNE_OK;
}

cprune_status cprune_plan_query(const cprune_plan *plan, cprune_plan_info *out) {
    if (!plan || !out) return CPRUNE_ERR_INVALID_ARG;
    *out = plan->info;
    return CPRUNE_OK;
}

cprune_status cprune_plan_release(cprune_plan *plan) {
    if (!plan) return CPRUNE_ERR_INVALID_ARG;
    PlanCache &c = cache();
    std::lock_guard<std::mutex> lock(c.mu);
    if (plan->refs <= 0) return CPRUNE_ERR_INVALID_ARG;
    --plan->refs;
    return CPRUNE_OK;
}

cprune_status cprune_cache_clear(int *n_left) {
    PlanCache &c = cache();
    std::lock_guard<std::mutex> lock(c.mu);
    for (auto it = c.plans.begin(); it != c.plans.end();) {
        if (it->second->refs == 0) {
            delete it->second;
            it = c.plans.erase(it);
        } else {
            ++it;
        }
    }
    if (n_left) *n_left = (int)c.plans.size();
    return CPRUNE_OK;
}

cprune_status cprune_cache_stats(int *n_plans, long long *n_hits) {
    PlanCache &c = cache();
    std::lock_guard<std::mutex> lock(c.mu);
    if (n_plans) *n_plans = (int)c.plans.size();
    if (n_hits) *n_hits = c.hits;
    return CPRUNE_OK;
}

cprune_status cprune_task_run(cprune_plan *plan, const void *x, const void *w_packed, const float *b_packed,
                              const void *residual, void *y, void *workspace, void *stream) {
    return task_run_internal(plan, x, w_packed, b_packed, residual, y, workspace, (cudaStream_t)stream, false);
}

}  // extern "C"
