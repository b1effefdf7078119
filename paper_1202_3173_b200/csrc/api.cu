// C ABI of the library (declared in include/strassen_b200.h): argument checking, lazy device
// set-up, and replay of a plan's launch list on the caller's stream.
#include "strassen_b200.h"

#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "bilinear.h"
#include "kernels.h"
#include "plan.h"

using namespace strassen;

namespace {

thread_local std::string g_error;

int fail(int status, const std::string &msg)
{
    g_error = msg;
    return status;
}

int cuda_fail(cudaError_t e, const char *what)
{
    return fail(STRASSEN_CUDA_ERROR, std::string(what) + ": " + cudaGetErrorString(e));
}

struct TimedLaunch {
    int kind;
    cudaEvent_t start, stop;
};

}  // namespace

struct strassen_plan {
    PlanDesc d;
    int device = -1;
    int sm_count = 0;
    Node *d_tab = nullptr;
    double *ws = nullptr;
    size_t ws_bytes = 0;
    bool own_ws = false;
    double *stage[2][3] = {{nullptr, nullptr, nullptr}, {nullptr, nullptr, nullptr}};   // host entry point: A, B, C copies
    int stage_sets = 0;
    bool host_pipeline = false;           // STRASSEN_FLAG_HOST_PIPELINE
    cudaStream_t s_h2d = nullptr, s_cmp = nullptr, s_d2h = nullptr;
    cudaEvent_t ev_h2d[2] = {nullptr, nullptr}, ev_cmp[2] = {nullptr, nullptr}, ev_d2h[2] = {nullptr, nullptr};
    uint64_t host_calls = 0;
    bool timing = false;
    std::vector<TimedLaunch> pending;
    std::vector<cudaEvent_t> free_events;
    bool use_graph = false;               // STRASSEN_FLAG_CUDA_GRAPH
    cudaStream_t capture_stream = nullptr;
    cudaGraphExec_t graph_exec = nullptr;
    const void *graph_ptrs[4] = {nullptr, nullptr, nullptr, nullptr};   // A, B, C, workspace the graph was captured for
    bool scheme_vec = false;              // generic bilinear plan: every level size, leading dimension and stride is even
    double acc_ms[STRASSEN_K_COUNT] = {};
    int64_t launches[STRASSEN_K_COUNT] = {};
    int64_t launch_total = 0;
};

namespace {

// Kernel family (strassen_kernel_kind) a launch is counted and timed under.
int family(int op_kind)
{
    if (op_kind == OP_FORM2 || op_kind == OP_FORM3 || op_kind == OP_FORM2_ODD) return STRASSEN_K_FORM;
    if (op_kind == OP_RECOMBINE2 || op_kind == OP_RECOMBINE3 || op_kind == OP_RECOMBINE2_ODD) return STRASSEN_K_RECOMBINE;
    if (op_kind == OP_SCALE_IN || op_kind == OP_SCALE_OUT) return STRASSEN_K_SCALE;
    if (op_kind == OP_FUSED_STEP) return STRASSEN_K_FUSED_STEP;
    if (op_kind == OP_LINCOMB) return STRASSEN_K_LINCOMB;
    return op_kind;
}

int64_t extent_words(int64_t n, int64_t ld, int64_t stride, int64_t batch)
{
    return (batch - 1) * stride + (n - 1) * ld + n;
}

bool overlap(const double *x, int64_t xw, const double *y, int64_t yw)
{
    const uintptr_t x0 = reinterpret_cast<uintptr_t>(x), x1 = x0 + uintptr_t(xw) * 8;
    const uintptr_t y0 = reinterpret_cast<uintptr_t>(y), y1 = y0 + uintptr_t(yw) * 8;
    return x0 < y1 && y0 < x1;
}

cudaEvent_t take_event(strassen_plan *p)
{
    if (!p->free_events.empty()) {
        cudaEvent_t e = p->free_events.back();
        p->free_events.pop_back();
        return e;
    }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
}

// Wait for the timing events recorded so far, add their durations to the per-family sums and recycle the events.
int harvest_timings(strassen_plan *p)
{
    for (TimedLaunch &t : p->pending) {
        cudaError_t e = cudaEventSynchronize(t.stop);
        if (e != cudaSuccess) return cuda_fail(e, "cudaEventSynchronize");
        float ms = 0.f;
        e = cudaEventElapsedTime(&ms, t.start, t.stop);
        if (e != cudaSuccess) return cuda_fail(e, "cudaEventElapsedTime");
        p->acc_ms[t.kind] += double(ms);
        p->free_events.push_back(t.start);
        p->free_events.push_back(t.stop);
    }
    p->pending.clear();
    return STRASSEN_OK;
}

constexpr size_t kMaxPendingTimings = 1 << 16;   // event pairs kept before a timed call folds them into the sums

// First use on a device: node tables, SM count, workspace.
int ensure_device_state(strassen_plan *p, cudaStream_t stream)
{
    if (p->device < 0) {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
        int major = 0;
        e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute");
        if (major != 10)
            return fail(STRASSEN_CUDA_ERROR, "this library holds sm_100a code only; the current device is not a B200-class GPU");
        e = cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute");
        e = configure_gemm_kernels();       // opt-in to large dynamic shared memory, outside any capture
        if (e == cudaSuccess) e = configure_fused_step_kernels();
        if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute");
        p->device = dev;
    } else {
        // tables, workspace and staging buffers live on the device of the first call
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
        if (dev != p->device) {
            char buf[128];
            snprintf(buf, sizeof buf, "the plan was first used on device %d; the current device is %d", p->device, dev);
            return fail(STRASSEN_INVALID_ARG, buf);
        }
    }
    if (!p->d_tab) {
        const size_t bytes = p->d.nodes.size() * sizeof(Node);
        cudaError_t e = cudaMalloc(&p->d_tab, bytes);
        if (e != cudaSuccess) return cuda_fail(e, "cudaMalloc(node tables)");
        // In the call's own stream, then waited for: a plain cudaMemcpy from pageable memory may return while
        // its last DMA is still queued, and a kernel in a non-blocking stream is not ordered behind it.
        e = cudaMemcpyAsync(p->d_tab, p->d.nodes.data(), bytes, cudaMemcpyHostToDevice, stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
        if (e != cudaSuccess) {
            cudaFree(p->d_tab);
            p->d_tab = nullptr;
            return cuda_fail(e, "copying the node tables to the device");
        }
    }
    const size_t need = size_t(p->d.ws_words) * 8;
    if (need > 0 && !p->ws) {
        cudaError_t e = cudaMalloc(&p->ws, need);
        if (e != cudaSuccess) {
            cudaGetLastError();
            char buf[160];
            snprintf(buf, sizeof buf, "cudaMalloc of %zu workspace bytes failed: %s", need, cudaGetErrorString(e));
            return fail(STRASSEN_OUT_OF_MEMORY, buf);
        }
        p->ws_bytes = need;
        p->own_ws = true;
    }
    return STRASSEN_OK;
}

// Enqueue every launch of the plan on `stream` (optionally bracketed by timing events).
int enqueue_launches(strassen_plan *p, const Bases &bases, bool bases16, cudaStream_t stream, bool timed)
{
    int launched = 0;
    if (timed && p->pending.size() + p->d.launches.size() > kMaxPendingTimings) {
        // timing left on and never read: fold what has accumulated (waits for those launches) instead of growing
        const int rc = harvest_timings(p);
        if (rc != STRASSEN_OK) return rc;
    }
    for (const Launch &op : p->d.launches) {
        const bool vec = op.vec_ok && bases16;
        TimedLaunch t{family(op.kind), nullptr, nullptr};
        if (timed) {
            t.start = take_event(p);
            t.stop = take_event(p);
            cudaEventRecord(t.start, stream);
        }
        cudaError_t e = cudaSuccess;
        switch (op.kind) {
        case OP_FORM: e = launch_form(p->d_tab, op, bases, vec, stream, &launched); break;
        case OP_GEMM: e = launch_gemm(p->d_tab, op, bases, p->sm_count, stream, &launched); break;
        case OP_RECOMBINE: e = launch_recombine(p->d_tab, op, bases, vec, stream, &launched); break;
        case OP_FORM_ONE: e = launch_form_one(p->d_tab, op, bases, vec, stream, &launched); break;
        case OP_ACCUMULATE: e = launch_accumulate(p->d_tab, op, bases, vec, stream, &launched); break;
        case OP_PEEL: e = launch_peel(p->d_tab, op, bases, stream, &launched); break;
        case OP_FORM2: e = launch_form2(p->d_tab, op, bases, vec, stream, &launched); break;
        case OP_RECOMBINE2: e = launch_recombine2(p->d_tab, op, bases, vec, stream, &launched); break;
        case OP_FORM2_ODD: e = launch_form2_odd(p->d_tab, op, bases, stream, &launched); break;
        case OP_RECOMBINE2_ODD: e = launch_recombine2_odd(p->d_tab, op, bases, stream, &launched); break;
        case OP_FORM3: e = launch_form3(p->d_tab, op, bases, stream, &launched); break;
        case OP_RECOMBINE3: e = launch_recombine3(p->d_tab, op, bases, stream, &launched); break;
        case OP_LINCOMB: {
            // the linear combinations of a generic scheme take 16-byte accesses where the whole plan allows them
            const LinComb &lc = reinterpret_cast<const LinComb *>(p->d.lincombs.data())[op.j];
            e = launch_lincomb(p->d_tab, op, lc, bases, bases16 && p->scheme_vec, stream, &launched);
            break;
        }
        case OP_FUSED_STEP: e = launch_fused_step(p->d_tab, op, bases, p->sm_count, stream, &launched); break;
        case OP_SCALE_IN: e = launch_scale_in(p->d, bases, stream, &launched); break;
        case OP_SCALE_OUT: e = launch_scale_out(p->d, bases, stream, &launched); break;
        }
        if (timed) {
            cudaEventRecord(t.stop, stream);
            p->pending.push_back(t);
        }
        if (e != cudaSuccess) return cuda_fail(e, "kernel launch");
    }
    return STRASSEN_OK;
}

// STRASSEN_FLAG_CUDA_GRAPH: the launch list is captured once per (A, B, C, workspace) into a CUDA graph on
// an internal stream and replayed on the caller's stream with a single launch.
int replay_graph(strassen_plan *p, const Bases &bases, bool bases16, cudaStream_t stream)
{
    bool same = p->graph_exec != nullptr;
    for (int i = 0; i < 4; ++i) same = same && p->graph_ptrs[i] == bases.p[i];
    if (!same) {
        if (!p->capture_stream) {
            cudaError_t e = cudaStreamCreateWithFlags(&p->capture_stream, cudaStreamNonBlocking);
            if (e != cudaSuccess) return cuda_fail(e, "cudaStreamCreate(capture)");
        }
        if (p->graph_exec) {
            cudaGraphExecDestroy(p->graph_exec);
            p->graph_exec = nullptr;
        }
        cudaError_t e = cudaStreamBeginCapture(p->capture_stream, cudaStreamCaptureModeThreadLocal);
        if (e != cudaSuccess) return cuda_fail(e, "cudaStreamBeginCapture");
        const int rc = enqueue_launches(p, bases, bases16, p->capture_stream, false);
        cudaGraph_t graph = nullptr;
        e = cudaStreamEndCapture(p->capture_stream, &graph);
        if (rc != STRASSEN_OK) {
            if (graph) cudaGraphDestroy(graph);
            return rc;
        }
        if (e != cudaSuccess || !graph) return cuda_fail(e, "cudaStreamEndCapture");
        e = cudaGraphInstantiate(&p->graph_exec, graph, 0);
        cudaGraphDestroy(graph);
        if (e != cudaSuccess) {
            p->graph_exec = nullptr;
            return cuda_fail(e, "cudaGraphInstantiate");
        }
        for (int i = 0; i < 4; ++i) p->graph_ptrs[i] = bases.p[i];
    }
    cudaError_t e = cudaGraphLaunch(p->graph_exec, stream);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGraphLaunch");
    return STRASSEN_OK;
}

strassen_plan *create(const strassen_options &o)
{
    g_error.clear();
    const int64_t n = o.n, cutoff = o.cutoff;
    const int64_t batch = o.batch == 0 ? 1 : o.batch;
    if (n < 1 || cutoff < 0 || batch < 1) {
        fail(STRASSEN_INVALID_ARG, "n and batch must be positive, cutoff non-negative");
        return nullptr;
    }
    if (n > (int64_t(1) << 30)) {
        fail(STRASSEN_INVALID_ARG, "n exceeds 2^30");
        return nullptr;
    }
    strassen_plan *p = new (std::nothrow) strassen_plan;
    if (!p) {
        fail(STRASSEN_OUT_OF_MEMORY, "out of host memory");
        return nullptr;
    }
    PlanDesc &d = p->d;
    d.n = n; d.cutoff = cutoff; d.batch = batch;
    d.lda = o.lda ? o.lda : n; d.ldb = o.ldb ? o.ldb : n; d.ldc = o.ldc ? o.ldc : n;
    d.stride_a = o.stride_a ? o.stride_a : d.lda * n;
    d.stride_b = o.stride_b ? o.stride_b : d.ldb * n;
    d.stride_c = o.stride_c ? o.stride_c : d.ldc * n;
    const int64_t ldmax = 0x7fffffff;
    if (d.lda < n || d.ldb < n || d.ldc < n || d.lda > ldmax || d.ldb > ldmax || d.ldc > ldmax) {
        fail(STRASSEN_INVALID_ARG, "leading dimensions must be >= n and fit 31 bits");
        delete p;
        return nullptr;
    }
    if (d.stride_a < 0 || d.stride_b < 0 || (batch > 1 && d.stride_c < (n - 1) * d.ldc + n)) {
        fail(STRASSEN_INVALID_ARG, "batch members of C must not overlap; strides must be non-negative");
        delete p;
        return nullptr;
    }
    d.fused_step = (o.flags & STRASSEN_FLAG_NO_FUSED_STEP) ? 2 : (o.flags & STRASSEN_FLAG_FUSED_STEP) ? 1 : 0;
    d.no_dfs_fold = (o.flags & STRASSEN_FLAG_NO_DFS_FOLD) != 0;
    d.max_fused_levels = (o.flags & STRASSEN_FLAG_SINGLE_LEVEL_PASSES) ? 1 : (o.flags & STRASSEN_FLAG_TWO_LEVEL_PASSES) ? 2 : 3;
    p->use_graph = (o.flags & STRASSEN_FLAG_CUDA_GRAPH) != 0;
    p->host_pipeline = (o.flags & STRASSEN_FLAG_HOST_PIPELINE) != 0;
    d.scale_inside = (o.flags & STRASSEN_FLAG_SCALE_INSIDE) != 0;
    d.scale_outside = (o.flags & STRASSEN_FLAG_SCALE_OUTSIDE) != 0;
    const bool want_auto = !o.schedule || strcmp(o.schedule, "auto") == 0;
    size_t budget = o.workspace_budget_bytes;
    if (want_auto && budget == 0 && (cutoff == 0 || n > cutoff)) {
        size_t free_b = 0, total_b = 0;
        cudaError_t e = cudaMemGetInfo(&free_b, &total_b);
        if (e != cudaSuccess) {
            cudaGetLastError();
            fail(STRASSEN_CUDA_ERROR, std::string("schedule \"auto\" without a workspace budget needs a CUDA device: ") +
                                          cudaGetErrorString(e));
            delete p;
            return nullptr;
        }
        const size_t margin = size_t(1) << 30;
        budget = free_b > margin ? free_b - margin : 0;
    }
    if (cutoff == 0 && want_auto) {
        // number of steps and interleaving by the cost model, among everything that fits the budget; bases
        // below 256 are left out: there the passes are latency-bound and the model, built on rates, is too kind
        if (!model_choice(n, batch, int64_t(budget / 8), 256, d.fused_step, &d.sizes, &d.schedule)) {
            fail(STRASSEN_WORKSPACE_TOO_SMALL, "no plan fits the workspace budget");
            delete p;
            return nullptr;
        }
    } else if (cutoff == 0) {
        // the schedule string fixes the number of steps
        const size_t steps = strlen(o.schedule);
        d.sizes.assign(1, n);
        while (d.sizes.size() <= steps && d.sizes.back() >= 2) d.sizes.push_back(d.sizes.back() / 2);
        if (d.sizes.size() != steps + 1) {
            fail(STRASSEN_BAD_SCHEDULE, "the schedule has more steps than n can be halved");
            delete p;
            return nullptr;
        }
    } else {
        d.sizes = level_sizes(n, cutoff);
    }
    d.cutoff = d.sizes.back();
    const size_t L = d.sizes.size() - 1;
    if (cutoff == 0 && want_auto) {
        // schedule chosen above
    } else if (want_auto) {
        if (!lm_schedule(d.sizes, batch, int64_t(budget / 8), &d.schedule)) {
            fail(STRASSEN_WORKSPACE_TOO_SMALL, "even the all-DFS schedule does not fit the workspace budget");
            delete p;
            return nullptr;
        }
    } else {
        d.schedule = o.schedule;
        if (d.schedule.size() != L) {
            char buf[128];
            snprintf(buf, sizeof buf, "schedule has %zu characters but the plan has %zu levels", d.schedule.size(), L);
            fail(STRASSEN_BAD_SCHEDULE, buf);
            delete p;
            return nullptr;
        }
        for (char c : d.schedule)
            if (c != 'B' && c != 'D') {
                fail(STRASSEN_BAD_SCHEDULE, "schedule characters must be 'B' or 'D'");
                delete p;
                return nullptr;
            }
        if (o.workspace_budget_bytes &&
            size_t(actual_workspace_words(d.sizes, d.schedule, batch)) * 8 > o.workspace_budget_bytes) {
            fail(STRASSEN_WORKSPACE_TOO_SMALL, "the schedule needs more workspace than the budget allows");
            delete p;
            return nullptr;
        }
    }
    const std::string err = build_plan(&d);
    if (!err.empty()) {
        fail(STRASSEN_INVALID_ARG, err);
        delete p;
        return nullptr;
    }
    for (const Launch &op : d.launches) {
        const int k = op.kind == OP_SCALE_IN ? scale_launches(d, true) : op.kind == OP_SCALE_OUT ? scale_launches(d, false)
                                                                                                : launches_of(op);
        p->launches[family(op.kind)] += k;
        p->launch_total += k;
    }
    return p;
}

// A plan for a generic <n0, n0, n0; q> scheme: the same handle type, its own level rule (sizes divide by n0, no
// peeling) and launch list.
strassen_plan *create_scheme(const strassen_options &o, const Scheme &s)
{
    g_error.clear();
    const std::string bad = validate_scheme(s);
    if (!bad.empty()) {
        fail(STRASSEN_INVALID_ARG, "not a matrix-multiplication scheme: " + bad);
        return nullptr;
    }
    const int64_t n = o.n, batch = o.batch == 0 ? 1 : o.batch;
    if (n < 1 || o.cutoff < 1 || batch < 1 || n > (int64_t(1) << 30)) {
        fail(STRASSEN_INVALID_ARG, "n, cutoff and batch must be positive (n at most 2^30)");
        return nullptr;
    }
    if (o.flags & ~int64_t(STRASSEN_FLAG_CUDA_GRAPH | STRASSEN_FLAG_HOST_PIPELINE)) {
        fail(STRASSEN_INVALID_ARG, "generic schemes take only the CUDA_GRAPH and HOST_PIPELINE flags");
        return nullptr;
    }
    strassen_plan *p = new (std::nothrow) strassen_plan;
    if (!p) {
        fail(STRASSEN_OUT_OF_MEMORY, "out of host memory");
        return nullptr;
    }
    PlanDesc &d = p->d;
    d.n = n; d.cutoff = o.cutoff; d.batch = batch;
    d.lda = o.lda ? o.lda : n; d.ldb = o.ldb ? o.ldb : n; d.ldc = o.ldc ? o.ldc : n;
    d.stride_a = o.stride_a ? o.stride_a : d.lda * n;
    d.stride_b = o.stride_b ? o.stride_b : d.ldb * n;
    d.stride_c = o.stride_c ? o.stride_c : d.ldc * n;
    const int64_t ldmax = 0x7fffffff;
    auto bail = [&](int status, const std::string &msg) {
        fail(status, msg);
        delete p;
        return static_cast<strassen_plan *>(nullptr);
    };
    if (d.lda < n || d.ldb < n || d.ldc < n || d.lda > ldmax || d.ldb > ldmax || d.ldc > ldmax)
        return bail(STRASSEN_INVALID_ARG, "leading dimensions must be >= n and fit 31 bits");
    if (d.stride_a < 0 || d.stride_b < 0 || (batch > 1 && d.stride_c < (n - 1) * d.ldc + n))
        return bail(STRASSEN_INVALID_ARG, "batch members of C must not overlap; strides must be non-negative");
    d.sizes = scheme_level_sizes(n, o.cutoff, s.n0);
    if (d.sizes.empty())
        return bail(STRASSEN_INVALID_ARG, "a generic scheme needs every level size above the cutoff to be divisible by n0 (no peeling)");
    d.cutoff = d.sizes.back();
    const size_t L = d.sizes.size() - 1;
    const bool want_auto = !o.schedule || strcmp(o.schedule, "auto") == 0;
    if (want_auto) {
        size_t budget = o.workspace_budget_bytes;
        if (budget == 0 && L > 0) {
            size_t free_b = 0, total_b = 0;
            if (cudaMemGetInfo(&free_b, &total_b) != cudaSuccess) {
                cudaGetLastError();
                return bail(STRASSEN_CUDA_ERROR, "schedule \"auto\" without a workspace budget needs a CUDA device");
            }
            budget = free_b > (size_t(1) << 30) ? free_b - (size_t(1) << 30) : 0;
        }
        bool found = false;       // Limited-Memory rule: the fewest leading DFS steps, then BFS steps only
        for (size_t ell = 0; ell <= L && !found; ++ell) {
            const std::string sched = std::string(ell, 'D') + std::string(L - ell, 'B');
            const int64_t w = scheme_workspace_words(s, d.sizes, sched, batch);
            if (w >= 0 && size_t(w) <= budget / 8) {
                d.schedule = sched;
                found = true;
            }
        }
        if (!found) return bail(STRASSEN_WORKSPACE_TOO_SMALL, "even the all-DFS schedule does not fit the workspace budget");
    } else {
        d.schedule = o.schedule;
        if (d.schedule.size() != L) return bail(STRASSEN_BAD_SCHEDULE, "the schedule must have one character per level");
        for (char c : d.schedule)
            if (c != 'B' && c != 'D') return bail(STRASSEN_BAD_SCHEDULE, "schedule characters must be 'B' or 'D'");
        if (o.workspace_budget_bytes && size_t(scheme_workspace_words(s, d.sizes, d.schedule, batch)) * 8 > o.workspace_budget_bytes)
            return bail(STRASSEN_WORKSPACE_TOO_SMALL, "the schedule needs more workspace than the budget allows");
    }
    const std::string err = build_scheme_plan(&d, s);
    if (!err.empty()) return bail(STRASSEN_INVALID_ARG, err);
    p->use_graph = (o.flags & STRASSEN_FLAG_CUDA_GRAPH) != 0;
    p->host_pipeline = (o.flags & STRASSEN_FLAG_HOST_PIPELINE) != 0;
    p->scheme_vec = ((d.lda | d.ldb | d.ldc | d.stride_a | d.stride_b | d.stride_c) & 1) == 0;
    for (size_t i = 0; i < d.sizes.size(); ++i) p->scheme_vec = p->scheme_vec && (i == 0 || d.sizes[i] % 2 == 0);
    for (const Launch &op : d.launches) {
        const int k = launches_of(op);
        p->launches[family(op.kind)] += k;
        p->launch_total += k;
    }
    return p;
}

}  // namespace

namespace strassen {
void set_last_error(const char *msg) { g_error = msg ? msg : ""; }
}  // namespace strassen

extern "C" {

strassen_plan *strassen_plan_create(int64_t n, int64_t cutoff, const char *schedule)
{
    strassen_options o;
    memset(&o, 0, sizeof o);
    o.n = n; o.cutoff = cutoff; o.schedule = schedule;
    return create(o);
}

strassen_plan *strassen_plan_create_ex(const strassen_options *opt)
{
    if (!opt) {
        fail(STRASSEN_INVALID_ARG, "options pointer is NULL");
        return nullptr;
    }
    return create(*opt);
}

strassen_plan *strassen_plan_create_scheme(const strassen_options *opt, const strassen_scheme *scheme)
{
    if (!opt || !scheme || !scheme->u || !scheme->v || !scheme->w) {
        fail(STRASSEN_INVALID_ARG, "options, scheme and its three tables must be non-NULL");
        return nullptr;
    }
    if (scheme->n0 < 2 || scheme->n0 > 4 || scheme->q < 1 || scheme->q > kMaxSchemeProducts) {
        fail(STRASSEN_INVALID_ARG, "a scheme needs 2 <= n0 <= 4 and 1 <= q <= 64");
        return nullptr;
    }
    Scheme s;
    s.n0 = scheme->n0; s.q = scheme->q;
    const size_t cells = size_t(s.q) * s.n0 * s.n0;
    s.u.assign(scheme->u, scheme->u + cells);
    s.v.assign(scheme->v, scheme->v + cells);
    s.w.assign(scheme->w, scheme->w + cells);
    return create_scheme(*opt, s);
}

strassen_plan *strassen_plan_create_named_scheme(const strassen_options *opt, const char *name)
{
    Scheme s;
    if (!opt || !name || !builtin_scheme(name, &s)) {
        fail(STRASSEN_INVALID_ARG, "options must be non-NULL and the name one of \"classical\", \"strassen\", \"winograd\"");
        return nullptr;
    }
    return create_scheme(*opt, s);
}

int strassen_scheme_check(const strassen_scheme *scheme)
{
    g_error.clear();
    if (!scheme || !scheme->u || !scheme->v || !scheme->w) return fail(STRASSEN_INVALID_ARG, "scheme and its three tables must be non-NULL");
    if (scheme->n0 < 2 || scheme->n0 > 4 || scheme->q < 1 || scheme->q > kMaxSchemeProducts)
        return fail(STRASSEN_INVALID_ARG, "a scheme needs 2 <= n0 <= 4 and 1 <= q <= 64");
    Scheme s;
    s.n0 = scheme->n0; s.q = scheme->q;
    const size_t cells = size_t(s.q) * s.n0 * s.n0;
    s.u.assign(scheme->u, scheme->u + cells);
    s.v.assign(scheme->v, scheme->v + cells);
    s.w.assign(scheme->w, scheme->w + cells);
    const std::string bad = validate_scheme(s);
    if (!bad.empty()) return fail(STRASSEN_INVALID_ARG, bad);
    return STRASSEN_OK;
}

int strassen_dgemm(strassen_plan *p, const double *A, const double *B, double *C, void *stream_v)
{
    g_error.clear();
    if (!p || !A || !B || !C) return fail(STRASSEN_INVALID_ARG, "plan, A, B and C must be non-NULL");
    const uintptr_t bits = reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(B) | reinterpret_cast<uintptr_t>(C);
    if (bits & 7) return fail(STRASSEN_MISALIGNED, "A, B and C must be 8-byte aligned");
    const PlanDesc &d = p->d;
    const int64_t wa = extent_words(d.n, d.lda, d.stride_a, d.batch), wb = extent_words(d.n, d.ldb, d.stride_b, d.batch),
                  wc = extent_words(d.n, d.ldc, d.stride_c, d.batch);
    if (overlap(C, wc, A, wa) || overlap(C, wc, B, wb)) return fail(STRASSEN_ALIAS, "C overlaps A or B");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const int rc = ensure_device_state(p, stream);
    if (rc != STRASSEN_OK) return rc;
    if (p->ws && d.ws_words > 0) {
        const int64_t ww = d.ws_words;
        if (overlap(p->ws, ww, A, wa) || overlap(p->ws, ww, B, wb) || overlap(p->ws, ww, C, wc))
            return fail(STRASSEN_ALIAS, "the workspace overlaps A, B or C");
    }
    Bases bases;
    bases.p[BASE_A] = const_cast<double *>(A);
    bases.p[BASE_B] = const_cast<double *>(B);
    bases.p[BASE_C] = C;
    bases.p[BASE_WS] = p->ws;
    const bool bases16 = ((bits | reinterpret_cast<uintptr_t>(p->ws)) & 15) == 0;
    if (p->use_graph && !p->timing) return replay_graph(p, bases, bases16, stream);
    return enqueue_launches(p, bases, bases16, stream, p->timing);
}

int strassen_dgemm_host(strassen_plan *p, const double *hA, const double *hB, double *hC, void *stream_v)
{
    g_error.clear();
    if (!p || !hA || !hB || !hC) return fail(STRASSEN_INVALID_ARG, "plan, A, B and C must be non-NULL");
    const PlanDesc &d = p->d;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const size_t bytes[3] = {size_t(extent_words(d.n, d.lda, d.stride_a, d.batch)) * 8,
                             size_t(extent_words(d.n, d.ldb, d.stride_b, d.batch)) * 8,
                             size_t(extent_words(d.n, d.ldc, d.stride_c, d.batch)) * 8};
    if (p->stage_sets == 0) {
        // one set of device copies; a second one (pipelined mode) if the device has room for it
        const int want = p->host_pipeline ? 2 : 1;
        for (int s = 0; s < want; ++s) {
            cudaError_t e = cudaSuccess;
            for (int m = 0; m < 3 && e == cudaSuccess; ++m) e = cudaMalloc(&p->stage[s][m], bytes[m]);
            if (e != cudaSuccess) {
                cudaGetLastError();
                for (int m = 0; m < 3; ++m) {
                    cudaFree(p->stage[s][m]);
                    p->stage[s][m] = nullptr;
                }
                if (s == 0) return fail(STRASSEN_OUT_OF_MEMORY, std::string("staging buffers: ") + cudaGetErrorString(e));
                break;
            }
            p->stage_sets = s + 1;
        }
        if (p->host_pipeline) {
            cudaError_t e = cudaStreamCreateWithFlags(&p->s_h2d, cudaStreamNonBlocking);
            if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&p->s_cmp, cudaStreamNonBlocking);
            if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&p->s_d2h, cudaStreamNonBlocking);
            for (int s = 0; s < 2 && e == cudaSuccess; ++s) {
                e = cudaEventCreateWithFlags(&p->ev_h2d[s], cudaEventDisableTiming);
                if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->ev_cmp[s], cudaEventDisableTiming);
                if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->ev_d2h[s], cudaEventDisableTiming);
            }
            if (e != cudaSuccess) return cuda_fail(e, "creating the streams and events of the host pipeline");
        }
    }
    const size_t row = size_t(d.n) * 8;
    auto copy_in = [&](double *dst, int64_t ld, int64_t stride, const double *src, cudaStream_t st) -> cudaError_t {
        if (ld == d.n && stride == d.n * d.n)
            return cudaMemcpyAsync(dst, src, row * size_t(d.n) * size_t(d.batch), cudaMemcpyHostToDevice, st);
        for (int64_t b = 0; b < d.batch; ++b) {
            cudaError_t e = cudaMemcpy2DAsync(dst + b * stride, size_t(ld) * 8, src + b * d.n * d.n, row, row, size_t(d.n),
                                              cudaMemcpyHostToDevice, st);
            if (e != cudaSuccess) return e;
        }
        return cudaSuccess;
    };
    auto copy_out = [&](const double *src, cudaStream_t st) -> cudaError_t {
        if (d.ldc == d.n && d.stride_c == d.n * d.n)
            return cudaMemcpyAsync(hC, src, row * size_t(d.n) * size_t(d.batch), cudaMemcpyDeviceToHost, st);
        for (int64_t b = 0; b < d.batch; ++b) {
            cudaError_t e = cudaMemcpy2DAsync(hC + b * d.n * d.n, row, src + b * d.stride_c, size_t(d.ldc) * 8, row, size_t(d.n),
                                              cudaMemcpyDeviceToHost, st);
            if (e != cudaSuccess) return e;
        }
        return cudaSuccess;
    };
    if (!p->host_pipeline) {
        cudaError_t e = copy_in(p->stage[0][0], d.lda, d.stride_a, hA, stream);
        if (e == cudaSuccess) e = copy_in(p->stage[0][1], d.ldb, d.stride_b, hB, stream);
        if (e != cudaSuccess) return cuda_fail(e, "host-to-device copy");
        const int rc = strassen_dgemm(p, p->stage[0][0], p->stage[0][1], p->stage[0][2], stream_v);
        if (rc != STRASSEN_OK) return rc;
        e = copy_out(p->stage[0][2], stream);
        if (e != cudaSuccess) return cuda_fail(e, "device-to-host copy");
        return STRASSEN_OK;
    }
    // Pipelined over three plan-owned streams: the input copy of this call runs beside the previous call's
    // products and the result copy of the call before it.  An event that was never recorded does not block.
    const int s = int(p->host_calls++ % uint64_t(p->stage_sets));
    cudaStreamWaitEvent(p->s_h2d, p->ev_cmp[s], 0);             // the products that last read this set are done
    cudaError_t e = copy_in(p->stage[s][0], d.lda, d.stride_a, hA, p->s_h2d);
    if (e == cudaSuccess) e = copy_in(p->stage[s][1], d.ldb, d.stride_b, hB, p->s_h2d);
    if (e != cudaSuccess) return cuda_fail(e, "host-to-device copy");
    cudaEventRecord(p->ev_h2d[s], p->s_h2d);
    cudaStreamWaitEvent(p->s_cmp, p->ev_h2d[s], 0);
    cudaStreamWaitEvent(p->s_cmp, p->ev_d2h[s], 0);             // the result copy that last read this set's C is done
    const int rc = strassen_dgemm(p, p->stage[s][0], p->stage[s][1], p->stage[s][2], p->s_cmp);
    if (rc != STRASSEN_OK) return rc;
    cudaEventRecord(p->ev_cmp[s], p->s_cmp);
    cudaStreamWaitEvent(p->s_d2h, p->ev_cmp[s], 0);
    e = copy_out(p->stage[s][2], p->s_d2h);
    if (e != cudaSuccess) return cuda_fail(e, "device-to-host copy");
    cudaEventRecord(p->ev_d2h[s], p->s_d2h);
    cudaStreamWaitEvent(stream, p->ev_d2h[s], 0);               // the caller's stream sees the result
    return STRASSEN_OK;
}

void strassen_plan_destroy(strassen_plan *p)
{
    if (!p) return;
    for (TimedLaunch &t : p->pending) {
        cudaEventDestroy(t.start);
        cudaEventDestroy(t.stop);
    }
    for (cudaEvent_t e : p->free_events) cudaEventDestroy(e);
    if (p->graph_exec) cudaGraphExecDestroy(p->graph_exec);
    if (p->capture_stream) cudaStreamDestroy(p->capture_stream);
    if (p->d_tab) cudaFree(p->d_tab);
    if (p->own_ws && p->ws) cudaFree(p->ws);
    for (int s = 0; s < 2; ++s) {
        for (int m = 0; m < 3; ++m)
            if (p->stage[s][m]) cudaFree(p->stage[s][m]);
        if (p->ev_h2d[s]) cudaEventDestroy(p->ev_h2d[s]);
        if (p->ev_cmp[s]) cudaEventDestroy(p->ev_cmp[s]);
        if (p->ev_d2h[s]) cudaEventDestroy(p->ev_d2h[s]);
    }
    for (cudaStream_t st : {p->s_h2d, p->s_cmp, p->s_d2h})
        if (st) cudaStreamDestroy(st);
    delete p;
}

size_t strassen_plan_workspace_bytes(const strassen_plan *p) { return p ? size_t(p->d.ws_words) * 8 : 0; }

int strassen_plan_set_workspace(strassen_plan *p, void *device_ptr, size_t bytes)
{
    g_error.clear();
    if (!p) return fail(STRASSEN_INVALID_ARG, "plan is NULL");
    const size_t need = size_t(p->d.ws_words) * 8;
    if (need == 0) return STRASSEN_OK;
    if (!device_ptr) return fail(STRASSEN_INVALID_ARG, "workspace pointer is NULL");
    if (reinterpret_cast<uintptr_t>(device_ptr) & 255) return fail(STRASSEN_MISALIGNED, "workspace must be 256-byte aligned");
    if (bytes < need) {
        char buf[128];
        snprintf(buf, sizeof buf, "workspace of %zu bytes given, %zu needed", bytes, need);
        return fail(STRASSEN_WORKSPACE_TOO_SMALL, buf);
    }
    if (p->own_ws && p->ws) cudaFree(p->ws);
    p->ws = static_cast<double *>(device_ptr);
    p->ws_bytes = bytes;
    p->own_ws = false;       // a captured graph is re-captured on the next call (its workspace pointer differs)
    return STRASSEN_OK;
}

const char *strassen_plan_schedule(const strassen_plan *p) { return p ? p->d.schedule.c_str() : ""; }
int strassen_plan_levels(const strassen_plan *p) { return p ? int(p->d.sizes.size()) - 1 : -1; }
int64_t strassen_plan_level_size(const strassen_plan *p, int level)
{
    if (!p || level < 0 || size_t(level) >= p->d.sizes.size()) return -1;
    return p->d.sizes[size_t(level)];
}
int64_t strassen_plan_base_size(const strassen_plan *p) { return p ? p->d.sizes.back() : -1; }
int64_t strassen_plan_base_products(const strassen_plan *p)
{
    if (!p) return -1;
    int64_t c = 0;
    for (const Launch &op : p->d.launches)
        if (op.kind == OP_GEMM) c += op.count;
        else if (op.kind == OP_FUSED_STEP) c += 7 * op.count;     // the seven products of each parent, inside the kernel
    return c;
}
int64_t strassen_plan_launch_count(const strassen_plan *p) { return p ? p->launch_total : -1; }
int64_t strassen_plan_launches_of(const strassen_plan *p, int kind)
{
    if (!p || kind < 0 || kind >= STRASSEN_K_COUNT) return -1;
    return p->launches[kind];
}

double strassen_plan_pass_bytes(const strassen_plan *p)
{
    if (!p || p->d.scheme_n0) return -1.0;       // the model describes the Strassen-Winograd plans only
    return plan_model_parts(p->d.sizes, p->d.schedule, p->d.batch, p->d.fused_step).pass_bytes;
}

double strassen_plan_model_ms(const strassen_plan *p)
{
    if (!p || p->d.scheme_n0) return -1.0;
    return plan_model_ms(p->d.sizes, p->d.schedule, p->d.batch, p->d.fused_step);
}

size_t strassen_schedule_model_bytes(int64_t n, int64_t cutoff, int64_t batch, const char *schedule, int accounting)
{
    g_error.clear();
    if (n < 1 || cutoff < 1 || batch < 1 || !schedule) {
        fail(STRASSEN_INVALID_ARG, "n, cutoff, batch must be positive and schedule non-NULL");
        return 0;
    }
    const int64_t w = model_workspace_words(level_sizes(n, cutoff), schedule, batch, accounting);
    if (w < 0) {
        fail(STRASSEN_BAD_SCHEDULE, "schedule must have one 'B' or 'D' per level and accounting must be 15 or 21");
        return 0;
    }
    return size_t(w) * 8;
}

int strassen_plan_set_timing(strassen_plan *p, int enabled)
{
    if (!p) return fail(STRASSEN_INVALID_ARG, "plan is NULL");
    p->timing = enabled != 0;
    return STRASSEN_OK;
}

int strassen_plan_get_timings(strassen_plan *p, double *ms_out)
{
    g_error.clear();
    if (!p || !ms_out) return fail(STRASSEN_INVALID_ARG, "plan and output must be non-NULL");
    const int rc = harvest_timings(p);
    if (rc != STRASSEN_OK) return rc;
    for (int k = 0; k < STRASSEN_K_COUNT; ++k) {
        ms_out[k] = p->acc_ms[k];
        p->acc_ms[k] = 0.0;
    }
    return STRASSEN_OK;
}

int strassen_probe_fp64(int kind, int64_t iters, void *stream, double *tflops_out)
{
    g_error.clear();
    if (kind < 0 || kind > 4 || iters < 1 || !tflops_out) return fail(STRASSEN_INVALID_ARG, "kind in 0..4, iters >= 1, output non-NULL");
    cudaError_t e = probe_fp64(kind, iters, static_cast<cudaStream_t>(stream), tflops_out);
    if (e != cudaSuccess) return cuda_fail(e, "fp64 probe");
    return STRASSEN_OK;
}

const char *strassen_last_error(void) { return g_error.c_str(); }

}  // extern "C"
