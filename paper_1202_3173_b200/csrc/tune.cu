// strassen_autotune: measured choice of the number of Strassen steps and of the BFS/DFS
// interleaving (Section 5.4: every point of the paper's plot is tuned to the best interleaving
// pattern and the best total number of Strassen steps).  Brute force over the candidates that fit
// the caller's workspace, timed with CUDA events on the caller's stream, in the order of a cost
// model so that a time limit cuts off the unlikely ones.
#include "strassen_b200.h"

#include <cstdio>
#include <algorithm>
#include <cstring>
#include <string>
#include <vector>

#include <cuda_runtime.h>

#include "kernels.h"
#include "plan.h"

using namespace strassen;

namespace {

int tune_fail(int status, const std::string &msg)
{
    set_last_error(msg.c_str());
    return status;
}

}  // namespace

extern "C" int strassen_autotune(const strassen_tune_request *req, strassen_tune_entry *best, strassen_tune_entry *log,
                                 int log_capacity, int *log_count)
{
    set_last_error("");
    if (log_count) *log_count = 0;
    if (!req || !best) return tune_fail(STRASSEN_INVALID_ARG, "request and result must be non-NULL");
    if (!req->A || !req->B || !req->C) return tune_fail(STRASSEN_INVALID_ARG, "A, B and C must be non-NULL");
    const int64_t n = req->n, batch = req->batch == 0 ? 1 : req->batch;
    if (n < 1 || batch < 1) return tune_fail(STRASSEN_INVALID_ARG, "n and batch must be positive");
    if (req->workspace_bytes > 0 && !req->workspace) return tune_fail(STRASSEN_INVALID_ARG, "workspace is NULL");
    const int64_t min_base = req->min_base > 0 ? req->min_base : 128;
    const int reps = req->repetitions > 0 ? req->repetitions : 2;
    const double max_seconds = req->max_seconds > 0 ? req->max_seconds : 60.0;
    cudaStream_t stream = static_cast<cudaStream_t>(req->stream);

    cudaEvent_t e0 = nullptr, e1 = nullptr, wall0 = nullptr;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess || cudaEventCreate(&wall0) != cudaSuccess)
        return tune_fail(STRASSEN_CUDA_ERROR, "cudaEventCreate failed");
    cudaEventRecord(wall0, stream);

    memset(best, 0, sizeof *best);
    best->ms = -1.0;
    int tried = 0, status = STRASSEN_OK;
    bool out_of_time = false;
    // L Strassen steps <=> cutoff = size of level L (recursion continues while size > cutoff)
    std::vector<int64_t> sizes{n};
    while (sizes.back() / 2 >= min_base && sizes.size() <= 10) sizes.push_back(sizes.back() / 2);
    struct Candidate {
        int64_t cutoff;
        std::string sched;
        double model;
    };
    std::vector<Candidate> candidates;
    for (size_t L = 0; L < sizes.size(); ++L) {
        const std::vector<int64_t> chain(sizes.begin(), sizes.begin() + L + 1);
        for (unsigned mask = 0; mask < (1u << L); ++mask) {
            std::string sched(L, 'B');
            for (size_t i = 0; i < L; ++i)
                if (mask >> i & 1) sched[i] = 'D';
            const int64_t words = actual_workspace_words(chain, sched, batch);
            if (words < 0 || size_t(words) > req->workspace_bytes / 8) continue;       // does not fit the workspace
            candidates.push_back(Candidate{sizes[L], sched, plan_model_ms(chain, sched, batch, 0)});
        }
    }
    // most promising first, so that a search cut short by max_seconds has seen the likely winners
    std::stable_sort(candidates.begin(), candidates.end(), [](const Candidate &a, const Candidate &b) { return a.model < b.model; });
    for (const Candidate &cand : candidates) {
        if (out_of_time || status != STRASSEN_OK) break;
        {
            const int64_t cutoff = cand.cutoff;
            const std::string &sched = cand.sched;
            const size_t L = sched.size();
            strassen_options o;
            memset(&o, 0, sizeof o);
            o.n = n; o.cutoff = cutoff; o.schedule = sched.c_str(); o.batch = batch;
            o.workspace_budget_bytes = req->workspace_bytes ? req->workspace_bytes : 1;   // explicit schedules are checked against it
            strassen_plan *p = strassen_plan_create_ex(&o);
            if (!p) continue;                                   // does not fit the node tables
            if (strassen_plan_set_workspace(p, req->workspace, req->workspace_bytes) != STRASSEN_OK) {
                strassen_plan_destroy(p);
                continue;
            }
            double ms_best = -1.0;
            for (int r = 0; r <= reps; ++r) {                   // first run warms up (and uploads the tables)
                cudaEventRecord(e0, stream);
                status = strassen_dgemm(p, req->A, req->B, req->C, stream);
                cudaEventRecord(e1, stream);
                if (status != STRASSEN_OK || cudaEventSynchronize(e1) != cudaSuccess) {
                    if (status == STRASSEN_OK) status = tune_fail(STRASSEN_CUDA_ERROR, "a candidate failed on the device");
                    break;
                }
                float ms = 0.f;
                cudaEventElapsedTime(&ms, e0, e1);
                if (r > 0 && (ms_best < 0 || ms < ms_best)) ms_best = ms;
            }
            strassen_plan_destroy(p);
            if (status != STRASSEN_OK) break;
            ++tried;
            strassen_tune_entry ent;
            memset(&ent, 0, sizeof ent);
            ent.cutoff = cutoff; ent.levels = int(L); ent.ms = ms_best; ent.model_ms = cand.model;
            snprintf(ent.schedule, sizeof ent.schedule, "%s", sched.c_str());
            if (log && log_count && *log_count < log_capacity) log[(*log_count)++] = ent;
            if (best->ms < 0 || ms_best < best->ms) *best = ent;
            float wall = 0.f;
            cudaEventElapsedTime(&wall, wall0, e1);
            if (wall * 1e-3 > max_seconds) out_of_time = true;
        }
    }
    cudaEventDestroy(e0); cudaEventDestroy(e1); cudaEventDestroy(wall0);
    if (status != STRASSEN_OK) return status;
    if (tried == 0) return tune_fail(STRASSEN_WORKSPACE_TOO_SMALL, "no candidate fits the workspace");
    // leave C holding the product computed by the chosen plan
    strassen_options o;
    memset(&o, 0, sizeof o);
    o.n = n; o.cutoff = best->cutoff; o.schedule = best->schedule; o.batch = batch;
    strassen_plan *p = strassen_plan_create_ex(&o);
    if (!p) return STRASSEN_INVALID_ARG;
    status = strassen_plan_set_workspace(p, req->workspace, req->workspace_bytes);
    if (status == STRASSEN_OK) status = strassen_dgemm(p, req->A, req->B, req->C, stream);
    if (status == STRASSEN_OK && cudaStreamSynchronize(stream) != cudaSuccess)
        status = tune_fail(STRASSEN_CUDA_ERROR, "synchronising after the tuned run failed");
    strassen_plan_destroy(p);
    return status;
}
