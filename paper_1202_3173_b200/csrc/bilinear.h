// Any <n0, n0, n0; q> bilinear matrix-multiplication scheme run through the same BFS / DFS traversal
// (Section 6.6 "Parallelizing other algorithms": q linear combinations of the n0 x n0 blocks of A and of B,
// q products, C's blocks as linear combinations of those; BFS or DFS decides whether the q products of a
// step are materialised side by side or one after another).
#pragma once
#include <cstdint>
#include <string>
#include <vector>

#include "plan.h"

namespace strassen {

struct Scheme {
    int n0 = 0, q = 0;
    std::vector<int8_t> u, v;   // q x n0^2: T_j = sum_b u[j][b] A_b, S_j = sum_b v[j][b] B_b (b = n0 * block row + block column)
    std::vector<int8_t> w;      // n0^2 x q: C_b = sum_j w[b][j] Q_j
};

constexpr int kMaxSchemeBlocks = 16;    // n0 <= 4
constexpr int kMaxSchemeProducts = 64;
constexpr int kLinCombTerms = 16;       // inputs one launch of the linear-combination kernel adds up

// One launch of the linear-combination kernel over `count` parents.
struct LinComb {
    int32_t mode;         // 0: child.a = sum coef * block src of parent.a; 1: the same for b; 2: block `out` of parent.c (+)= sum coef * child[src].c
    int32_t nterms;
    int32_t out;          // mode 0 / 1: child index j within the parent's children; mode 2: block index of C
    int32_t accumulate;   // mode 2: add to what the block holds (later touches of a DFS step, or a second chunk of terms)
    int32_t children;     // children per parent in the child table (q for a BFS step, 1 for a DFS step)
    int32_t n0;
    int8_t coef[kLinCombTerms];
    int8_t src[kLinCombTerms];
};

// Empty string if the tables satisfy the bilinear identities of an n0 x n0 product (every C_b equals
// sum_k A_(i,k) B_(k,j)), else a description of the first violated one.
std::string validate_scheme(const Scheme &s);

// The built-in tables: "classical" (<2,2,2;8>, the recursive classical algorithm), "strassen" (<2,2,2;7>, the
// original 18-addition form), "winograd" (<2,2,2;7>, Appendix A written out without shared sub-sums).
bool builtin_scheme(const std::string &name, Scheme *out);

// Level sizes m_0 = n, m_{i+1} = m_i / n0 while m_i > cutoff; empty if some m_i is not divisible by n0.
std::vector<int64_t> scheme_level_sizes(int64_t n, int64_t cutoff, int n0);

// Workspace words of a schedule: per BFS parent the non-trivial T and S combinations and q products, per DFS
// parent one (T, S, Q) triple; rows padded like the Strassen-Winograd plans.  -1 if the schedule is malformed.
int64_t scheme_workspace_words(const Scheme &s, const std::vector<int64_t> &sizes, const std::string &sched, int64_t batch);

// Fill p->levels, nodes, launches, lincombs, ws_words from sizes / schedule / scheme.  Empty string or an error.
std::string build_scheme_plan(PlanDesc *p, const Scheme &s);

}  // namespace strassen
