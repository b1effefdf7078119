// Host side of the generic <n0, n0, n0; q> bilinear schemes (Section 6.6): table validation, the built-in
// tables, level sizes, workspace, node tables and the launch list.
#include "bilinear.h"

#include <cstdio>
#include <cstring>

namespace strassen {

namespace {

constexpr int64_t kPad = 32;
int64_t up(int64_t x, int64_t q) { return (x + q - 1) / q * q; }

// a combination that is exactly one block with coefficient +1 is used in place (a view), never copied
int trivial_block(const int8_t *row, int nb)
{
    int at = -1;
    for (int b = 0; b < nb; ++b) {
        if (row[b] == 0) continue;
        if (row[b] != 1 || at >= 0) return -1;
        at = b;
    }
    return at;
}

Operand block_of(const Operand &x, int b, int n0, int64_t hh)
{
    Operand r = x;
    r.off = x.off + int64_t(b / n0) * hh * int64_t(x.ld) + int64_t(b % n0) * hh;
    return r;
}

struct SchemeBuilder {
    PlanDesc *p;
    const Scheme &s;
    std::string err;
    std::vector<LinComb> ops;

    int64_t append(const std::vector<Node> &v)
    {
        const int64_t at = int64_t(p->nodes.size());
        if (at + int64_t(v.size()) > (int64_t(1) << 23)) {
            err = "recursion tree too large for the node tables (more than 2^23 nodes)";
            return -1;
        }
        p->nodes.insert(p->nodes.end(), v.begin(), v.end());
        return at;
    }

    void push_lincomb(const LinComb &lc, int level, int64_t ptab, int64_t ctab, int64_t count, int64_t m, int64_t hh)
    {
        Launch l{};
        l.kind = OP_LINCOMB; l.level = level; l.j = int32_t(ops.size());
        l.parent_tab = ptab; l.child_tab = ctab; l.count = count; l.m = m; l.h = hh;
        ops.push_back(lc);
        p->launches.push_back(l);
    }

    // T_j (side 0) or S_j (side 1) of every parent, unless it is a plain block
    void form(int side, int j, int children, int level, int64_t ptab, int64_t ctab, int64_t count, int64_t m, int64_t hh)
    {
        const int nb = s.n0 * s.n0;
        const int8_t *row = (side ? s.v : s.u).data() + size_t(j) * nb;
        if (trivial_block(row, nb) >= 0) return;
        LinComb lc{};
        lc.mode = side; lc.out = children == 1 ? 0 : j; lc.children = children; lc.n0 = s.n0;
        for (int b = 0; b < nb; ++b)
            if (row[b]) {
                lc.coef[lc.nterms] = row[b];
                lc.src[lc.nterms] = int8_t(b);
                ++lc.nterms;
            }
        push_lincomb(lc, level, ptab, ctab, count, m, hh);
    }

    void build(int level, int64_t tab, int64_t count)
    {
        if (!err.empty()) return;
        const int L = int(p->levels.size());
        if (level == L) {
            Launch g{};
            g.kind = OP_GEMM; g.level = level; g.j = -1; g.vec_ok = 1;
            g.parent_tab = tab; g.child_tab = -1; g.count = count; g.m = p->sizes[level];
            p->launches.push_back(g);
            return;
        }
        const LevelInfo &lv = p->levels[level];
        const int nb = s.n0 * s.n0, q = s.q;
        const int64_t hh = lv.h, mat = lv.mat_words, ldw = lv.ldw, N = count;
        // slots of the non-trivial combinations
        std::vector<int> tslot(q, -1), sslot(q, -1);
        int nt = 0, ns = 0;
        for (int j = 0; j < q; ++j) {
            if (trivial_block(s.u.data() + size_t(j) * nb, nb) < 0) tslot[j] = nt++;
            if (trivial_block(s.v.data() + size_t(j) * nb, nb) < 0) sslot[j] = ns++;
        }
        if (lv.mode == 'B') {
            const int64_t t_base = lv.ws_off, s_base = t_base + N * nt * mat, q_base = s_base + N * ns * mat;
            std::vector<Node> kids(size_t(N) * q, Node{});
            for (int64_t par = 0; par < N; ++par) {
                const Node nd = p->nodes[tab + par];
                for (int j = 0; j < q; ++j) {
                    Node &k = kids[size_t(par) * q + j];
                    const int ta = trivial_block(s.u.data() + size_t(j) * nb, nb), tb = trivial_block(s.v.data() + size_t(j) * nb, nb);
                    k.a = ta >= 0 ? block_of(nd.a, ta, s.n0, hh) : Operand{t_base + (par * nt + tslot[j]) * mat, int32_t(ldw), BASE_WS};
                    k.b = tb >= 0 ? block_of(nd.b, tb, s.n0, hh) : Operand{s_base + (par * ns + sslot[j]) * mat, int32_t(ldw), BASE_WS};
                    k.c = Operand{q_base + (par * q + j) * mat, int32_t(ldw), BASE_WS};
                }
            }
            const int64_t ctab = append(kids);
            if (ctab < 0) return;
            for (int j = 0; j < q; ++j) {
                form(0, j, q, level, tab, ctab, N, lv.m, hh);
                form(1, j, q, level, tab, ctab, N, lv.m, hh);
            }
            build(level + 1, ctab, N * q);
            if (!err.empty()) return;
            for (int b = 0; b < nb; ++b) {      // C_b = sum_j w[b][j] Q_j, at most kLinCombTerms products per launch
                LinComb lc{};
                lc.mode = 2; lc.out = b; lc.children = q; lc.n0 = s.n0;
                for (int j = 0; j < q; ++j) {
                    const int8_t c = s.w[size_t(b) * q + j];
                    if (!c) continue;
                    if (lc.nterms == kLinCombTerms) {
                        push_lincomb(lc, level, tab, ctab, N, lv.m, hh);
                        lc.nterms = 0;
                        lc.accumulate = 1;
                    }
                    lc.coef[lc.nterms] = c;
                    lc.src[lc.nterms] = int8_t(j);
                    ++lc.nterms;
                }
                push_lincomb(lc, level, tab, ctab, N, lv.m, hh);
            }
        } else {
            const int64_t t_base = lv.ws_off, s_base = t_base + N * mat, q_base = s_base + N * mat;
            std::vector<char> touched(size_t(nb), 0);
            for (int j = 0; j < q; ++j) {
                std::vector<Node> kids(size_t(N), Node{});
                const int ta = trivial_block(s.u.data() + size_t(j) * nb, nb), tb = trivial_block(s.v.data() + size_t(j) * nb, nb);
                for (int64_t par = 0; par < N; ++par) {
                    const Node nd = p->nodes[tab + par];
                    Node &k = kids[size_t(par)];
                    k.a = ta >= 0 ? block_of(nd.a, ta, s.n0, hh) : Operand{t_base + par * mat, int32_t(ldw), BASE_WS};
                    k.b = tb >= 0 ? block_of(nd.b, tb, s.n0, hh) : Operand{s_base + par * mat, int32_t(ldw), BASE_WS};
                    k.c = Operand{q_base + par * mat, int32_t(ldw), BASE_WS};
                }
                const int64_t ctab = append(kids);
                if (ctab < 0) return;
                form(0, j, 1, level, tab, ctab, N, lv.m, hh);
                form(1, j, 1, level, tab, ctab, N, lv.m, hh);
                build(level + 1, ctab, N);
                if (!err.empty()) return;
                for (int b = 0; b < nb; ++b) {      // the contribution of Q_j to every block of C that uses it
                    const int8_t c = s.w[size_t(b) * q + j];
                    if (!c) continue;
                    LinComb lc{};
                    lc.mode = 2; lc.out = b; lc.children = 1; lc.n0 = s.n0; lc.nterms = 1;
                    lc.coef[0] = c; lc.src[0] = 0;
                    lc.accumulate = touched[size_t(b)];
                    touched[size_t(b)] = 1;
                    push_lincomb(lc, level, tab, ctab, N, lv.m, hh);
                }
            }
        }
    }
};

}  // namespace

std::string validate_scheme(const Scheme &s)
{
    if (s.n0 < 2 || s.n0 * s.n0 > kMaxSchemeBlocks) return "n0 must be 2, 3 or 4";
    if (s.q < 1 || s.q > kMaxSchemeProducts) return "q must be 1..64";
    const int nb = s.n0 * s.n0, n0 = s.n0;
    if (int(s.u.size()) != s.q * nb || int(s.v.size()) != s.q * nb || int(s.w.size()) != nb * s.q) return "table sizes do not match n0 and q";
    // coefficient of A_(a,b) B_(c,d) in C_(e,f) must be 1 where b = c, a = e, d = f and 0 elsewhere
    for (int ab = 0; ab < nb; ++ab)
        for (int cd = 0; cd < nb; ++cd)
            for (int ef = 0; ef < nb; ++ef) {
                long sum = 0;
                for (int j = 0; j < s.q; ++j) sum += long(s.u[size_t(j) * nb + ab]) * s.v[size_t(j) * nb + cd] * s.w[size_t(ef) * s.q + j];
                const int a = ab / n0, b = ab % n0, c = cd / n0, d = cd % n0, e = ef / n0, f = ef % n0;
                const long want = (b == c && a == e && d == f) ? 1 : 0;
                if (sum != want) {
                    char buf[160];
                    snprintf(buf, sizeof buf, "the tables give coefficient %ld (not %ld) to A(%d,%d) B(%d,%d) in C(%d,%d)", sum, want, a, b, c, d, e, f);
                    return buf;
                }
            }
    for (int b = 0; b < nb; ++b) {
        bool any = false;
        for (int j = 0; j < s.q; ++j) any = any || s.w[size_t(b) * s.q + j];
        if (!any) return "a block of C receives no product";
    }
    return "";
}

bool builtin_scheme(const std::string &name, Scheme *out)
{
    Scheme s;
    s.n0 = 2;
    const int nb = 4;
    auto rows = [&](std::vector<int8_t> &t, std::initializer_list<std::initializer_list<int>> r) {
        for (const auto &row : r)
            for (int x : row) t.push_back(int8_t(x));
    };
    // blocks: 0 = X11, 1 = X12, 2 = X21, 3 = X22
    if (name == "classical") {
        // C11 = A11 B11 + A12 B21, C12 = A11 B12 + A12 B22, C21 = A21 B11 + A22 B21, C22 = A21 B12 + A22 B22
        s.q = 8;
        rows(s.u, {{1,0,0,0},{0,1,0,0},{1,0,0,0},{0,1,0,0},{0,0,1,0},{0,0,0,1},{0,0,1,0},{0,0,0,1}});
        rows(s.v, {{1,0,0,0},{0,0,1,0},{0,1,0,0},{0,0,0,1},{1,0,0,0},{0,0,1,0},{0,1,0,0},{0,0,0,1}});
        rows(s.w, {{1,1,0,0,0,0,0,0},{0,0,1,1,0,0,0,0},{0,0,0,0,1,1,0,0},{0,0,0,0,0,0,1,1}});
    } else if (name == "strassen") {
        // M1 = (A11+A22)(B11+B22)  M2 = (A21+A22) B11  M3 = A11 (B12-B22)  M4 = A22 (B21-B11)  M5 = (A11+A12) B22
        // M6 = (A21-A11)(B11+B12)  M7 = (A12-A22)(B21+B22)
        // C11 = M1+M4-M5+M7  C12 = M3+M5  C21 = M2+M4  C22 = M1-M2+M3+M6
        s.q = 7;
        rows(s.u, {{1,0,0,1},{0,0,1,1},{1,0,0,0},{0,0,0,1},{1,1,0,0},{-1,0,1,0},{0,1,0,-1}});
        rows(s.v, {{1,0,0,1},{1,0,0,0},{0,1,0,-1},{-1,0,1,0},{0,0,0,1},{1,1,0,0},{0,0,1,1}});
        rows(s.w, {{1,0,0,1,-1,0,1},{0,0,1,0,1,0,0},{0,1,0,1,0,0,0},{1,-1,1,0,0,1,0}});
    } else if (name == "winograd") {
        // Appendix A with the shared sub-sums written out: T3 = A21+A22-A11, T5 = A11+A12-A21-A22, S3 = B11-B12+B22,
        // S6 = B11-B12-B21+B22; C12 = Q0+Q2+Q3+Q5, C21 = Q0+Q3+Q4-Q6, C22 = Q0+Q2+Q3+Q4
        s.q = 7;
        rows(s.u, {{1,0,0,0},{0,1,0,0},{0,0,1,1},{-1,0,1,1},{1,0,-1,0},{1,1,-1,-1},{0,0,0,1}});
        rows(s.v, {{1,0,0,0},{0,0,1,0},{-1,1,0,0},{1,-1,0,1},{0,-1,0,1},{0,0,0,1},{1,-1,-1,1}});
        rows(s.w, {{1,1,0,0,0,0,0},{1,0,1,1,0,1,0},{1,0,0,1,1,0,-1},{1,0,1,1,1,0,0}});
    } else {
        return false;
    }
    (void)nb;
    *out = s;
    return true;
}

std::vector<int64_t> scheme_level_sizes(int64_t n, int64_t cutoff, int n0)
{
    std::vector<int64_t> m{n};
    while (m.back() > cutoff) {
        if (m.back() % n0) return {};
        m.push_back(m.back() / n0);
    }
    return m;
}

int64_t scheme_workspace_words(const Scheme &s, const std::vector<int64_t> &sizes, const std::string &sched, int64_t batch)
{
    if (sched.size() + 1 != sizes.size()) return -1;
    const int nb = s.n0 * s.n0;
    int nt = 0, ns = 0;
    for (int j = 0; j < s.q; ++j) {
        nt += trivial_block(s.u.data() + size_t(j) * nb, nb) < 0;
        ns += trivial_block(s.v.data() + size_t(j) * nb, nb) < 0;
    }
    int64_t words = 0, live = batch;
    for (size_t i = 0; i < sched.size(); ++i) {
        if (sched[i] != 'B' && sched[i] != 'D') return -1;
        const int64_t hh = sizes[i + 1], mat = up(hh * up(hh, 4), kPad);
        const int64_t per = sched[i] == 'B' ? nt + ns + s.q : 3;
        if (live > (int64_t(1) << 60) / (per * mat)) return int64_t(1) << 60;
        words += live * per * mat;
        if (sched[i] == 'B') live *= s.q;
        if (live > (int64_t(1) << 40)) return int64_t(1) << 60;
    }
    return words;
}

std::string build_scheme_plan(PlanDesc *p, const Scheme &s)
{
    const int L = int(p->sizes.size()) - 1;
    if (int(p->schedule.size()) != L) return "schedule does not match the number of levels";
    p->levels.clear(); p->nodes.clear(); p->launches.clear(); p->lincombs.clear();
    const int nb = s.n0 * s.n0;
    int nt = 0, ns = 0;
    for (int j = 0; j < s.q; ++j) {
        nt += trivial_block(s.u.data() + size_t(j) * nb, nb) < 0;
        ns += trivial_block(s.v.data() + size_t(j) * nb, nb) < 0;
    }
    int64_t live = p->batch, off = 0;
    for (int i = 0; i < L; ++i) {
        LevelInfo lv{};
        lv.m = p->sizes[i]; lv.h = p->sizes[i + 1];
        lv.ldw = up(lv.h, 4); lv.mat_words = up(lv.h * lv.ldw, kPad);
        lv.parents = live; lv.ws_off = off; lv.mode = p->schedule[i]; lv.peel = false;
        off += live * (lv.mode == 'B' ? nt + ns + s.q : 3) * lv.mat_words;
        if (lv.mode == 'B') live *= s.q;
        if (live > (int64_t(1) << 23)) return "recursion tree too large for the node tables (more than 2^23 nodes)";
        p->levels.push_back(lv);
    }
    p->ws_words = off;
    p->scheme_n0 = s.n0; p->scheme_q = s.q;
    std::vector<Node> top(size_t(p->batch), Node{});
    for (int64_t b = 0; b < p->batch; ++b) {
        top[size_t(b)].a = Operand{b * p->stride_a, int32_t(p->lda), BASE_A};
        top[size_t(b)].b = Operand{b * p->stride_b, int32_t(p->ldb), BASE_B};
        top[size_t(b)].c = Operand{b * p->stride_c, int32_t(p->ldc), BASE_C};
    }
    SchemeBuilder bld{p, s, {}, {}};
    const int64_t tab = bld.append(top);
    if (tab < 0) return bld.err;
    bld.build(0, tab, p->batch);
    p->lincombs.resize(bld.ops.size() * sizeof(LinComb));
    if (!bld.ops.empty()) memcpy(p->lincombs.data(), bld.ops.data(), p->lincombs.size());
    return bld.err;
}

}  // namespace strassen
