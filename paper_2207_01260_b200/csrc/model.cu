// Whole-model runner: the aggregate of a network's tasks enqueued back to back on one stream
// (paper Sec. 3.1: the model is the aggregate of its tasks' programs and is timed as a whole),
// optionally replayed as a CUDA graph so that one replay costs one host call.
#include <map>
#include <vector>

#include "common.cuh"
#include "plan.h"

struct ModelTensor {
    int n = 0, h = 0, w = 0, c = 0, c_pad = 0;
    size_t offset = 0, bytes = 0;
    bool defined = false;
};

struct cprune_model {
    int N, H, W, C;
    std::vector<cprune_task_desc> tasks;
    std::map<int, ModelTensor> tensors;
    char *arena = nullptr;
    size_t arena_bytes = 0;
    char *workspace = nullptr;
    size_t workspace_bytes = 0;
    int classes = 0;
    int launches = 0;
    // captured launch sequences: slot 2 serves cprune_model_run, slots 0 and 1 the two device-side
    // input buffers of cprune_model_run_host
    struct GraphSlot {
        cudaGraphExec_t exec = nullptr;
        const float *x = nullptr;
        float *logits = nullptr;
        cudaStream_t stream = nullptr;
    } graphs[3];
    cudaStream_t capture_stream = nullptr;   // private stream the launch sequence is recorded on
    // host-buffer path: double-buffered device copies of the input and of the logits
    float *host_x[2] = {nullptr, nullptr};
    float *host_logits[2] = {nullptr, nullptr};
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t copied[2] = {nullptr, nullptr}, done[2] = {nullptr, nullptr};
    unsigned long long host_calls = 0;
};

namespace cprune {

static size_t align256(size_t v) { return (v + 255) / 256 * 256; }

static void *tensor_ptr(const cprune_model *m, int id) {
    auto it = m->tensors.find(id);
    return it == m->tensors.end() ? nullptr : (void *)(m->arena + it->second.offset);
}

static cprune_status enqueue_chain(cprune_model *m, const float *x, float *logits, cudaStream_t st);

// The kernels of one pass are launched as a chain: each may start while its predecessor drains (see common.cuh).
static cprune_status enqueue(cprune_model *m, const float *x, float *logits, cudaStream_t st) {
    set_chain_launch(true);
    cprune_status s = enqueue_chain(m, x, logits, st);
    set_chain_launch(false);
    return s;
}

// True when the model's input is read by its first task only and that task is a stem that works on a regrouped
// input: the float32 image is then cast and regrouped in one pass and the bf16 NHWC copy is never written.
static bool stem_reads_image_directly(const cprune_model *m) {
    if (m->tasks.empty()) return false;
    const cprune_task_desc &d0 = m->tasks[0];
    if (d0.op != CPRUNE_OP_CONV || d0.in != 0 || !d0.plan || !d0.plan->patch || !d0.plan->narrow) return false;
    for (size_t t = 1; t < m->tasks.size(); ++t)
        if (m->tasks[t].in == 0 || m->tasks[t].res == 0) return false;
    return true;
}

static cprune_status enqueue_chain(cprune_model *m, const float *x, float *logits, cudaStream_t st) {
    const bool direct = stem_reads_image_directly(m);
    cprune_status s = direct ? regroup_stem_input(m->tasks[0].plan, x, 1, stem_scratch(m->tasks[0].plan, m->workspace), st)
                             : cprune_cast_input(x, (size_t)m->N * m->H * m->W, m->C, tensor_ptr(m, 0), st);
    if (s != CPRUNE_OK) return s;
    for (size_t t = 0; t < m->tasks.size(); ++t) {
        const cprune_task_desc &d = m->tasks[t];
        const ModelTensor &in = m->tensors[d.in];
        void *pin = tensor_ptr(m, d.in);
        const bool last = t + 1 == m->tasks.size();
        void *pout = last ? (void *)logits : tensor_ptr(m, d.out);
        switch (d.op) {
            case CPRUNE_OP_CONV:
                s = task_run_internal(d.plan, pin, d.w, d.b, d.res >= 0 ? tensor_ptr(m, d.res) : nullptr, pout, m->workspace, st,
                                      t == 0 && direct);
                break;
            case CPRUNE_OP_BLOCK:
                s = cprune_block_run(d.block, pin, d.w, d.b, pout, m->workspace, st);
                break;
            case CPRUNE_OP_MAXPOOL:
                s = cprune_maxpool(pin, in.n, in.h, in.w, in.c, d.p0, d.p1, d.p2, pout, st);
                break;
            case CPRUNE_OP_GAP:
                s = cprune_global_avgpool(pin, in.n, in.h, in.w, in.c, pout, st);
                break;
            case CPRUNE_OP_FC:
                s = cprune_fc(pin, in.n, d.p0, d.w, d.b, d.p1, d.p2, last ? 1 : 0, pout, st);
                break;
            default:
                s = CPRUNE_ERR_INTERNAL;
        }
        if (s != CPRUNE_OK) return s;
    }
    return CPRUNE_OK;
}

}  // namespace cprune

using namespace cprune;

extern "C" {

cprune_status cprune_model_create(int N, int H, int W, int C, const cprune_task_desc *tasks, int n_tasks,
                                  cprune_model **out) {
    if (!out) return CPRUNE_ERR_INVALID_ARG;
    *out = nullptr;
    if (N <= 0 || H <= 0 || W <= 0 || C <= 0 || !tasks || n_tasks <= 0) return CPRUNE_ERR_INVALID_ARG;
    if (tasks[n_tasks - 1].op != CPRUNE_OP_FC) return CPRUNE_ERR_INVALID_ARG;
    cprune_model *m = new cprune_model();
    m->N = N; m->H = H; m->W = W; m->C = C;
    m->tasks.assign(tasks, tasks + n_tasks);
    ModelTensor t0;
    t0.n = N; t0.h = H; t0.w = W; t0.c = C; t0.c_pad = cprune_padded_channels(C); t0.defined = true;
    m->tensors[0] = t0;
    m->launches = 1;
    cprune_status st = CPRUNE_OK;
    for (int t = 0; t < n_tasks && st == CPRUNE_OK; ++t) {
        const cprune_task_desc &d = m->tasks[t];
        auto it = m->tensors.find(d.in);
        if (it == m->tensors.end() || d.out <= 0) { st = CPRUNE_ERR_INVALID_ARG; break; }
        const ModelTensor in = it->second;
        ModelTensor o;
        o.n = in.n; o.defined = true;
        switch (d.op) {
            case CPRUNE_OP_CONV: {
                if (!d.plan || !d.w || !d.b) { st = CPRUNE_ERR_INVALID_ARG; break; }
                const cprune_plan_info &i = d.plan->info;
                if (i.N != in.n || i.H != in.h || i.W != in.w || i.C != in.c) { st = CPRUNE_ERR_INVALID_ARG; break; }
                if ((d.plan->opts.residual != 0) != (d.res >= 0)) { st = CPRUNE_ERR_INVALID_ARG; break; }
                if (d.res >= 0) {
                    auto r = m->tensors.find(d.res);
                    if (r == m->tensors.end() || r->second.h != i.P || r->second.w != i.Q || r->second.c != i.K) {
                        st = CPRUNE_ERR_INVALID_ARG;
                        break;
                    }
                }
                o.h = i.out_h; o.w = i.out_w; o.c = i.K;
                if (i.workspace_bytes > m->workspace_bytes) m->workspace_bytes = i.workspace_bytes;
                m->launches += ((d.plan->opts.pool && !(i.kernel == CPRUNE_KERNEL_TENSOR && d.plan->fused_pool)) ? 2 : 1) + (d.plan->splits > 1 ? 1 : 0) +
                               ((d.plan->patch && d.plan->narrow) ? 1 : 0);
                break;
            }
            case CPRUNE_OP_BLOCK: {
                if (!d.block || !d.w || !d.b) { st = CPRUNE_ERR_INVALID_ARG; break; }
                cprune_block_info bi;
                if (cprune_block_query(d.block, &bi) != CPRUNE_OK || bi.N != in.n || bi.H != in.h || bi.W != in.w || bi.C_in != in.c) {
                    st = CPRUNE_ERR_INVALID_ARG;
                    break;
                }
                o.h = bi.H; o.w = bi.W; o.c = bi.C_out;
                if (bi.workspace_bytes > m->workspace_bytes) m->workspace_bytes = bi.workspace_bytes;
                m->launches += bi.splits > 1 ? 2 : 1;
                break;
            }
            case CPRUNE_OP_MAXPOOL:
                if (d.p0 <= 0 || d.p1 <= 0 || d.p2 < 0 || in.h + 2 * d.p2 < d.p0 || in.w + 2 * d.p2 < d.p0) {
                    st = CPRUNE_ERR_INVALID_ARG;
                    break;
                }
                o.h = (in.h + 2 * d.p2 - d.p0) / d.p1 + 1; o.w = (in.w + 2 * d.p2 - d.p0) / d.p1 + 1; o.c = in.c;
                m->launches += 1;
                break;
            case CPRUNE_OP_GAP:
                o.h = 1; o.w = 1; o.c = in.c;
                m->launches += 1;
                break;
            case CPRUNE_OP_FC:
                if (!d.w || !d.b || in.h * in.w != 1 || in.c != d.p0 || d.p1 <= 0) { st = CPRUNE_ERR_INVALID_ARG; break; }
                o.h = 1; o.w = 1; o.c = d.p1;
                m->launches += 1;
                if (t == n_tasks - 1) m->classes = d.p1;
                break;
            default:
                st = CPRUNE_ERR_INVALID_ARG;
        }
        if (st != CPRUNE_OK) break;
        o.c_pad = cprune_padded_channels(o.c);
        if (m->tensors.count(d.out)) { st = CPRUNE_ERR_INVALID_ARG; break; }   // single assignment
        m->tensors[d.out] = o;
    }
    if (st != CPRUNE_OK) { delete m; return st; }
    if (stem_reads_image_directly(m)) m->launches -= 1;     // one pass casts and regroups the image
    size_t off = 0;
    for (auto &kv : m->tensors) {
        kv.second.bytes = (size_t)kv.second.n * kv.second.h * kv.second.w * kv.second.c_pad * 2;
        kv.second.offset = off;
        off += align256(kv.second.bytes);
    }
    m->arena_bytes = off;
    cudaError_t e = cudaMalloc((void **)&m->arena, m->arena_bytes);
    if (e == cudaSuccess && m->workspace_bytes) e = cudaMalloc((void **)&m->workspace, m->workspace_bytes);
    if (e != cudaSuccess) {
        if (m->arena) cudaFree(m->arena);
        delete m;
        return cuda_fail(e, "cudaMalloc(model activations)");
    }
    *out = m;
    return CPRUNE_OK;
}

static cprune_status run_graph(cprune_model *m, int slot, const float *x, float *logits, cudaStream_t st) {
    cprune_model::GraphSlot &g = m->graphs[slot];
    if (g.exec && g.x == x && g.logits == logits && g.stream == st) {
        CPRUNE_CUDA_CHECK(cudaGraphLaunch(g.exec, st));
        return CPRUNE_OK;
    }
    if (g.exec) { cudaGraphExecDestroy(g.exec); g.exec = nullptr; }
    // first call for this (x, logits, stream): run eagerly (this also encodes tensor maps and sets
    // kernel attributes outside of any capture), then record the same sequence for later replays
    cprune_status s = enqueue(m, x, logits, st);
    if (s != CPRUNE_OK) return s;
    // the caller's stream may be the legacy default stream, which cannot be captured: record on a
    // private stream and replay the graph on the caller's
    if (!m->capture_stream) CPRUNE_CUDA_CHECK(cudaStreamCreateWithFlags(&m->capture_stream, cudaStreamNonBlocking));
    cudaGraph_t graph = nullptr;
    CPRUNE_CUDA_CHECK(cudaStreamBeginCapture(m->capture_stream, cudaStreamCaptureModeThreadLocal));
    s = enqueue(m, x, logits, m->capture_stream);
    cudaError_t e = cudaStreamEndCapture(m->capture_stream, &graph);
    if (s != CPRUNE_OK) { if (graph) cudaGraphDestroy(graph); return s; }
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamEndCapture");
    e = cudaGraphInstantiate(&g.exec, graph, 0);
    cudaGraphDestroy(graph);
    if (e != cudaSuccess) { g.exec = nullptr; return cuda_fail(e, "cudaGraphInstantiate"); }
    g.x = x; g.logits = logits; g.stream = st;
    return CPRUNE_OK;
}

cprune_status cprune_model_run(cprune_model *m, const float *x, float *logits, int use_graph, void *stream) {
    if (!m || !x || !logits) return CPRUNE_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (!use_graph) return enqueue(m, x, logits, st);
    return run_graph(m, 2, x, logits, st);
}

cprune_status cprune_model_run_host(cprune_model *m, const float *x_host, float *logits_host, void *stream) {
    if (!m || !x_host || !logits_host) return CPRUNE_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t x_bytes = (size_t)m->N * m->H * m->W * m->C * sizeof(float);
    const size_t l_bytes = (size_t)m->N * m->classes * sizeof(float);
    if (!m->copy_stream) {   // first call: set up the two device-side buffer pairs (allocates)
        CPRUNE_CUDA_CHECK(cudaStreamCreateWithFlags(&m->copy_stream, cudaStreamNonBlocking));
        for (int i = 0; i < 2; ++i) {
            CPRUNE_CUDA_CHECK(cudaMalloc((void **)&m->host_x[i], x_bytes));
            CPRUNE_CUDA_CHECK(cudaMalloc((void **)&m->host_logits[i], l_bytes));
            CPRUNE_CUDA_CHECK(cudaEventCreateWithFlags(&m->copied[i], cudaEventDisableTiming));
            CPRUNE_CUDA_CHECK(cudaEventCreateWithFlags(&m->done[i], cudaEventDisableTiming));
        }
    }
    const int slot = (int)(m->host_calls & 1);
    // the copy of this call's input may overlap the previous call's kernels; it only has to wait
    // until the call before that one has finished with the same device buffer
    if (m->host_calls >= 2) CPRUNE_CUDA_CHECK(cudaStreamWaitEvent(m->copy_stream, m->done[slot], 0));
    CPRUNE_CUDA_CHECK(cudaMemcpyAsync(m->host_x[slot], x_host, x_bytes, cudaMemcpyHostToDevice, m->copy_stream));
    CPRUNE_CUDA_CHECK(cudaEventRecord(m->copied[slot], m->copy_stream));
    CPRUNE_CUDA_CHECK(cudaStreamWaitEvent(st, m->copied[slot], 0));
    cprune_status s = run_graph(m, slot, m->host_x[slot], m->host_logits[slot], st);
    if (s != CPRUNE_OK) return s;
    CPRUNE_CUDA_CHECK(cudaMemcpyAsync(logits_host, m->host_logits[slot], l_bytes, cudaMemcpyDeviceToHost, st));
    CPRUNE_CUDA_CHECK(cudaEventRecord(m->done[slot], st));
    ++m->host_calls;
    return CPRUNE_OK;
}

cprune_status cprune_model_tensor(const cprune_model *m, int id, const void **ptr, int *n, int *h, int *w, int *c_pad) {
    if (!m) return CPRUNE_ERR_INVALID_ARG;
    auto it = m->tensors.find(id);
    if (it == m->tensors.end()) return CPRUNE_ERR_INVALID_ARG;
    if (ptr) *ptr = m->arena + it->second.offset;
    if (n) *n = it->second.n;
    if (h) *h = it->second.h;
    if (w) *w = it->second.w;
    if (c_pad) *c_pad = it->second.c_pad;
    return CPRUNE_OK;
}

cprune_status cprune_model_copy_tensor(const cprune_model *m, int id, void *dst, void *stream) {
    if (!m || !dst) return CPRUNE_ERR_INVALID_ARG;
    auto it = m->tensors.find(id);
    if (it == m->tensors.end()) return CPRUNE_ERR_INVALID_ARG;
    CPRUNE_CUDA_CHECK(cudaMemcpyAsync(dst, m->arena + it->second.offset, it->second.bytes, cudaMemcpyDeviceToDevice,
                                      (cudaStream_t)stream));
    return CPRUNE_OK;
}

int cprune_model_launches(const cprune_model *m) { return m ? m->launches : 0; }

cprune_status cprune_model_task_table(const cprune_model *m, cprune_task_entry *entries, int max_entries, int *n_entries) {
    if (!m || !n_entries || max_entries < 0 || (max_entries > 0 && !entries)) return CPRUNE_ERR_INVALID_ARG;
    std::vector<cprune_task_entry> table;
    for (size_t t = 0; t < m->tasks.size(); ++t) {
        const cprune_task_desc &d = m->tasks[t];
        if (d.op != CPRUNE_OP_CONV) continue;
        bool found = false;
        for (auto &e : table)
            if (e.plan == d.plan) { ++e.count; found = true; break; }
        if (!found) table.push_back(cprune_task_entry{d.plan, 1, (int)t});
    }
    *n_entries = (int)table.size();
    for (int j = 0; j < (int)table.size() && j < max_entries; ++j) entries[j] = table[j];
    return CPRUNE_OK;
}

cprune_status cprune_model_time_tasks(cprune_model *m, int reps, double *ms, void *stream) {
    if (!m || !ms || reps < 1) return CPRUNE_ERR_INVALID_ARG;
    int n = 0;
    cprune_status s = cprune_model_task_table(m, nullptr, 0, &n);
    if (s != CPRUNE_OK) return s;
    std::vector<cprune_task_entry> table(n);
    s = cprune_model_task_table(m, table.data(), n, &n);
    if (s != CPRUNE_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    CPRUNE_CUDA_CHECK(cudaEventCreate(&e0));
    CPRUNE_CUDA_CHECK(cudaEventCreate(&e1));
    for (int j = 0; j < n && s == CPRUNE_OK; ++j) {
        const cprune_task_desc &d = m->tasks[table[j].first_task];
        void *pin = tensor_ptr(m, d.in), *pout = tensor_ptr(m, d.out);
        const void *res = d.res >= 0 ? tensor_ptr(m, d.res) : nullptr;
        for (int r = 0; r <= reps && s == CPRUNE_OK; ++r) {
            if (r == 1 && cudaEventRecord(e0, st) != cudaSuccess) s = CPRUNE_ERR_CUDA;   // run 0 is the untimed one
            if (s == CPRUNE_OK) s = task_run_internal(d.plan, pin, d.w, d.b, res, pout, m->workspace, st, false);
        }
        if (s != CPRUNE_OK) break;
        float t = 0.f;
        if (cudaEventRecord(e1, st) != cudaSuccess || cudaEventSynchronize(e1) != cudaSuccess ||
            cudaEventElapsedTime(&t, e0, e1) != cudaSuccess) { s = cuda_fail(cudaGetLastError(), "task timing"); break; }
        ms[j] = (double)t / reps;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    return s;
}

cprune_status cprune_model_destroy(cprune_model *m) {
    if (!m) return CPRUNE_ERR_INVALID_ARG;
    for (auto &g : m->graphs)
        if (g.exec) cudaGraphExecDestroy(g.exec);
    if (m->capture_stream) cudaStreamDestroy(m->capture_stream);
    if (m->copy_stream) cudaStreamDestroy(m->copy_stream);
    for (int i = 0; i < 2; ++i) {
        if (m->host_x[i]) cudaFree(m->host_x[i]);
        if (m->host_logits[i]) cudaFree(m->host_logits[i]);
        if (m->copied[i]) cudaEventDestroy(m->copied[i]);
        if (m->done[i]) cudaEventDestroy(m->done[i]);
    }
    if (m->arena) cudaFree(m->arena);
    if (m->workspace) cudaFree(m->workspace);
    delete m;
    return CPRUNE_OK;
}

}  // extern "C"
