// Host-side check of the planner, built with AddressSanitizer and UBSan by tests/test_plan_sanitized.py:
// for a sweep of sizes, cutoffs, batches and B/D strings (and the generic bilinear schemes) every operand of
// every node must lie inside the allocation it names, workspace operands inside the planned workspace, and no
// two operands that one launch group writes may overlap.  Prints "ok <plans> <nodes>" or the first violation.
#include <cstdio>
#include <cstdlib>
#include <string>
#include <vector>

#include "bilinear.h"
#include "plan.h"

using namespace strassen;

static long long g_plans = 0, g_nodes = 0;

static bool inside(const Operand &x, int64_t rows, int64_t cols, int64_t limit, const char *what, const PlanDesc &d)
{
    const int64_t last = x.off + (rows - 1) * int64_t(x.ld) + cols;
    if (x.off < 0 || x.ld < cols || last > limit) {
        printf("FAIL n=%lld sched=%s: %s operand off=%lld ld=%d rows=%lld cols=%lld exceeds %lld\n", (long long)d.n, d.schedule.c_str(), what,
               (long long)x.off, x.ld, (long long)rows, (long long)cols, (long long)limit);
        return false;
    }
    return true;
}

static int64_t extent(int64_t n, int64_t ld, int64_t stride, int64_t batch) { return (batch - 1) * stride + (n - 1) * ld + n; }

static bool check(const PlanDesc &d)
{
    ++g_plans;
    const int64_t lim[4] = {extent(d.n, d.lda, d.stride_a, d.batch), extent(d.n, d.ldb, d.stride_b, d.batch),
                            extent(d.n, d.ldc, d.stride_c, d.batch), d.ws_words};
    for (const Launch &op : d.launches) {
        if (op.kind != OP_GEMM) continue;
        for (int64_t i = 0; i < op.count; ++i) {          // the leaves: operands of size m x m
            const Node &nd = d.nodes[size_t(op.parent_tab + i)];
            ++g_nodes;
            if (!inside(nd.a, op.m, op.m, lim[nd.a.base], "leaf A", d) || !inside(nd.b, op.m, op.m, lim[nd.b.base], "leaf B", d) ||
                !inside(nd.c, op.m, op.m, lim[nd.c.base], "leaf C", d))
                return false;
            if (nd.a.base == BASE_C || nd.b.base == BASE_C) {
                printf("FAIL: a leaf reads the result matrix\n");
                return false;
            }
        }
        if (op.sibling_tab > 0) {       // the leaves are the sevens of children of these parents, whose quadrants the thin products read
            if (op.count % 7 != 0 || op.sibling_tab - 1 + op.count / 7 > int64_t(d.nodes.size()) || op.sibling_tab - 1 + op.count / 7 > op.parent_tab) {
                printf("FAIL n=%lld sched=%s: sibling parents out of the node table\n", (long long)d.n, d.schedule.c_str());
                return false;
            }
            for (int64_t i = 0; i < op.count / 7; ++i) {
                const Node &par = d.nodes[size_t(op.sibling_tab - 1 + i)];
                if (!inside(par.a, 2 * op.m, 2 * op.m, lim[par.a.base], "sibling parent A", d) ||
                    !inside(par.b, 2 * op.m, 2 * op.m, lim[par.b.base], "sibling parent B", d))
                    return false;
            }
        }
        // products of one launch must not overlap each other
        std::vector<std::pair<int64_t, int64_t>> spans;
        for (int64_t i = 0; i < op.count; ++i) {
            const Node &nd = d.nodes[size_t(op.parent_tab + i)];
            if (nd.c.base == BASE_WS) spans.push_back({nd.c.off, nd.c.off + (op.m - 1) * int64_t(nd.c.ld) + op.m});
        }
        std::sort(spans.begin(), spans.end());
        for (size_t i = 1; i < spans.size(); ++i)
            if (spans[i].first < spans[i - 1].second) {
                printf("FAIL n=%lld sched=%s: two products of one launch overlap in the workspace\n", (long long)d.n, d.schedule.c_str());
                return false;
            }
    }
    return true;
}

int main()
{
    unsigned long long state = 12345;
    auto rnd = [&](int mod) {
        state = state * 6364136223846793005ULL + 1442695040888963407ULL;
        return int((state >> 33) % unsigned(mod));
    };
    for (int trial = 0; trial < 400; ++trial) {
        PlanDesc d;
        d.n = 1 + rnd(900);
        d.batch = 1 + rnd(3);
        d.lda = d.n + rnd(3); d.ldb = d.n + rnd(3); d.ldc = d.n + rnd(3);
        d.stride_a = d.lda * d.n + rnd(5); d.stride_b = d.ldb * d.n; d.stride_c = d.ldc * d.n + rnd(7);
        const int64_t cutoff = 1 + rnd(int(d.n));
        d.sizes = level_sizes(d.n, cutoff > d.n / 40 ? cutoff : d.n / 40 + 1);
        d.schedule.clear();
        for (size_t i = 0; i + 1 < d.sizes.size(); ++i) d.schedule.push_back(rnd(2) ? 'B' : 'D');
        d.max_fused_levels = 1 + rnd(3);
        d.fused_step = rnd(3);
        d.no_dfs_fold = rnd(2);
        d.scale_outside = rnd(4) == 0;
        const std::string err = build_plan(&d);
        if (!err.empty()) {
            printf("FAIL build_plan: %s\n", err.c_str());
            return 1;
        }
        if (d.ws_words < actual_workspace_words(d.sizes, d.schedule, d.batch)) {
            printf("FAIL: planned workspace below the model's\n");
            return 1;
        }
        if (!check(d)) return 1;
    }
    for (const char *name : {"classical", "strassen", "winograd"}) {
        Scheme s;
        if (!builtin_scheme(name, &s) || !validate_scheme(s).empty()) {
            printf("FAIL: built-in scheme %s does not validate\n", name);
            return 1;
        }
        for (int trial = 0; trial < 40; ++trial) {
            PlanDesc d;
            const int L = rnd(4);
            d.n = int64_t(1 + rnd(9)) << L;
            d.batch = 1 + rnd(2);
            d.lda = d.ldb = d.ldc = d.n;
            d.stride_a = d.stride_b = d.stride_c = d.n * d.n;
            d.sizes = scheme_level_sizes(d.n, d.n >> L, s.n0);
            d.schedule.clear();
            for (size_t i = 0; i + 1 < d.sizes.size(); ++i) d.schedule.push_back(rnd(2) ? 'B' : 'D');
            const std::string err = build_scheme_plan(&d, s);
            if (!err.empty()) {
                printf("FAIL build_scheme_plan: %s\n", err.c_str());
                return 1;
            }
            if (d.ws_words != scheme_workspace_words(s, d.sizes, d.schedule, d.batch)) {
                printf("FAIL: scheme workspace differs from its model\n");
                return 1;
            }
            if (!check(d)) return 1;
        }
    }
    printf("ok %lld %lld\n", g_plans, g_nodes);
    return 0;
}
