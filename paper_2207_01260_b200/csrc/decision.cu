// Host-side steps of the method around the tasks (paper Sec. 3.3 and Sec. 3.5): how many filters to prune
// so that a task keeps the structure of its program, what the pruned task is expected to cost, and in which
// order a model's tasks are tried.  Nothing here launches a kernel.
#include <algorithm>
#include <numeric>
#include <vector>

#include "common.cuh"
#include "plan.h"

namespace {

long long gcd_ll(long long a, long long b) {
    while (b) { long long t = a % b; a = b; b = t; }
    return a;
}

// smallest slice of one iterator: (product of its factors) / (largest factor), in filters
long long smallest_slice(const int *split, int unit) {
    long long prod = 1;
    int largest = 1;
    for (int j = 0; j < 2; ++j) {
        const int f = split[j] < 1 ? 1 : split[j];
        prod *= f;
        largest = std::max(largest, f);
    }
    return (long long)unit * (prod / largest);
}

}  // namespace

extern "C" {

cprune_status cprune_prune_step(const cprune_plan *plan, int *step) {
    if (!plan || !step) return CPRUNE_ERR_INVALID_ARG;
    const cprune_plan_info &i = plan->info;
    const long long a = smallest_slice(i.split_compute, i.unit_compute);
    const long long b = smallest_slice(i.split_store, i.unit_store);
    if (a <= 0 || b <= 0) return CPRUNE_ERR_INTERNAL;
    *step = (int)(a / gcd_ll(a, b) * b);
    return CPRUNE_OK;
}

cprune_status cprune_task_estimate(const cprune_plan *plan, int k_new, double *est_us) {
    if (!plan || !est_us || k_new < 1) return CPRUNE_ERR_INVALID_ARG;
    const cprune_plan_info &i = plan->info;
    const bool depthwise = i.groups > 1;
    // a depthwise task loses the input channel with the filter; a dense task keeps its input
    cprune_plan *other = nullptr;
    cprune_status st = cprune_task_plan(i.N, depthwise ? k_new : i.C, i.H, i.W, k_new, i.R, i.S, i.stride, i.pad,
                                        depthwise ? k_new : 1, &plan->opts, &other);
    if (st != CPRUNE_OK) return st;
    *est_us = other->info.est_us;
    return cprune_plan_release(other);
}

cprune_status cprune_task_order(const double *times, const int *counts, int n, int *order) {
    if (n < 0 || (n > 0 && (!times || !counts || !order))) return CPRUNE_ERR_INVALID_ARG;
    std::vector<int> idx(n);
    std::iota(idx.begin(), idx.end(), 0);
    std::stable_sort(idx.begin(), idx.end(), [&](int a, int b) { return times[a] * counts[a] > times[b] * counts[b]; });
    for (int j = 0; j < n; ++j) order[j] = idx[j];
    return CPRUNE_OK;
}

}  // extern "C"
