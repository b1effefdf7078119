// Host-side planning: level sizes, BFS/DFS schedule against a workspace budget
// (Limited-Memory rule, Section 3.4), workspace carve-up, node tables and the launch list.
#include "plan.h"

#include "kernels.h"

#include <limits>

namespace strassen {

namespace {

constexpr int64_t kMaxNodes = int64_t(1) << 23;   // table entries (48 B each)
constexpr int64_t kPadWords = 32;                 // workspace matrices start on 256-byte boundaries

int64_t round_up(int64_t x, int64_t q) { return (x + q - 1) / q * q; }

bool sched_ok(const std::vector<int64_t> &sizes, const std::string &s)
{
    if (s.size() + 1 != sizes.size()) return false;
    for (char c : s)
        if (c != 'B' && c != 'D') return false;
    return true;
}

// The seven operand pairs of a node (Appendix A): which A-side / B-side operand of child j
// is a plain quadrant (index 0..3 = X11, X12, X21, X22) and which is a computed sum (-1).
constexpr int kTQuad[7] = {0, 1, -1, -1, -1, -1, 3};   // T0=A11 T1=A12 T6=A22
constexpr int kSQuad[7] = {0, 2, -1, -1, -1, 3, -1};   // S0=B11 S1=B21 S5=B22
constexpr int kTSlot[7] = {-1, -1, 0, 1, 2, 3, -1};    // T2..T5 -> slot 0..3
constexpr int kSSlot[7] = {-1, -1, 0, 1, 2, -1, 3};    // S2,S3,S4,S6 -> slot 0..3

Operand quadrant(const Operand &x, int q, int64_t h)
{
    Operand r = x;
    r.off = x.off + (q & 1 ? h : 0) + (q & 2 ? h * int64_t(x.ld) : 0);
    return r;
}

Operand ws_mat(int64_t off, int64_t ldw) { return Operand{off, int32_t(ldw), BASE_WS}; }

bool even(const Operand &x) { return (x.off & 1) == 0 && (x.ld & 1) == 0; }

struct Builder {
    PlanDesc *p;
    std::string err;

    int64_t append(const std::vector<Node> &v)
    {
        const int64_t at = int64_t(p->nodes.size());
        if (at + int64_t(v.size()) > kMaxNodes) {
            err = "recursion tree too large for the node tables (more than 2^23 nodes)";
            return -1;
        }
        p->nodes.insert(p->nodes.end(), v.begin(), v.end());
        return at;
    }

    // The 7 children of each of the N nodes at p->nodes[tab ..) for a BFS step at level `lv`.
    std::vector<Node> bfs_children(int64_t tab, int64_t N, const LevelInfo &lv) const
    {
        const int64_t h = lv.h, mat = lv.mat_words, ldw = lv.ldw;
        std::vector<Node> kids(static_cast<size_t>(N) * 7, Node{});
        const int64_t t_base = lv.ws_off, s_base = lv.ws_off + N * 4 * mat, q_base = lv.ws_off + N * 8 * mat;
        for (int64_t q = 0; q < N; ++q) {
            const Node nd = p->nodes[tab + q];
            for (int j = 0; j < 7; ++j) {
                Node &k = kids[size_t(q) * 7 + j];
                k.a = kTQuad[j] >= 0 ? quadrant(nd.a, kTQuad[j], h) : ws_mat(t_base + (q * 4 + kTSlot[j]) * mat, ldw);
                k.b = kSQuad[j] >= 0 ? quadrant(nd.b, kSQuad[j], h) : ws_mat(s_base + (q * 4 + kSSlot[j]) * mat, ldw);
                k.c = ws_mat(q_base + (q * 7 + j) * mat, ldw);
            }
        }
        return kids;
    }

    // the deepest level as one fused kernel takes no part in the multi-level passes above it
    bool fused_last() const
    {
        if (p->levels.empty()) return false;
        const LevelInfo &lv = p->levels.back();
        return fused_step_chosen(p->fused_step, p->schedule, lv.h, lv.parents);
    }
    int group_size(int level, bool *odd_pair) const
    {
        const std::string sched = fused_last() ? p->schedule.substr(0, p->schedule.size() - 1) : p->schedule;
        return fused_group_size(p->sizes, sched, level, p->max_fused_levels, odd_pair);
    }

    // nodes of `level` are p->nodes[tab .. tab + count); siblings: 1 + the index of their parents' first node where they
    // are the complete, consecutive sets of seven children of parents whose operands are in memory in full (a BFS step
    // of its own, or the pair with an odd lower member), 0 otherwise
    void build(int level, int64_t tab, int64_t count, int64_t siblings = 0)
    {
        if (!err.empty()) return;
        const int L = int(p->levels.size());
        if (level == L) {
            Launch g{};
            g.kind = OP_GEMM; g.level = level; g.j = -1; g.vec_ok = 1;
            g.parent_tab = tab; g.child_tab = -1; g.count = count;
            g.m = p->sizes[level]; g.h = 0;
            g.sibling_tab = siblings;
            p->launches.push_back(g);
            return;
        }
        const LevelInfo &lv = p->levels[level];
        const int64_t h = lv.h, mat = lv.mat_words, ldw = lv.ldw, N = count;
        // 16-byte accesses: what a recombination touches (the parents' C; their A and B only for the rank-one term of an
        // odd parent) is tracked apart from what a formation touches
        bool c_even = (h & 1) == 0, ab_even = (h & 1) == 0;
        for (int64_t q = 0; q < N; ++q) {
            const Node &nd = p->nodes[tab + q];
            c_even = c_even && even(nd.c);
            ab_even = ab_even && even(nd.a) && even(nd.b);
        }
        const bool parents_even = c_even && ab_even, recombine_even = c_even && (!lv.peel || ab_even);
        if (lv.mode == 'B' && level == L - 1 && fused_last()) {
            Launch f{};
            f.kind = OP_FUSED_STEP; f.level = level; f.j = -1; f.vec_ok = parents_even;
            f.parent_tab = tab; f.child_tab = -1; f.grand_tab = -1; f.count = N; f.m = lv.m; f.h = h;
            f.peel_fused = lv.peel;
            p->launches.push_back(f);
        } else if (lv.mode == 'B') {
            const int64_t ctab = append(bfs_children(tab, N, lv));
            if (ctab < 0) return;
            Launch f{};
            f.kind = OP_FORM; f.level = level; f.j = -1; f.vec_ok = parents_even;
            f.parent_tab = tab; f.child_tab = ctab; f.count = N; f.m = lv.m; f.h = h;
            f.grand_tab = -1;
            bool odd_pair = false;
            const int group = group_size(level, &odd_pair);
            if (group >= 2) {
                // several BFS levels in one pass: the sums of the intermediate levels are still written
                // (the operands below are views into them), their products are not
                const LevelInfo &lv2 = p->levels[level + 1];
                const int64_t gtab = append(bfs_children(ctab, N * 7, lv2));
                if (gtab < 0) return;
                f.grand_tab = gtab;
                f.reg.child_t = lv.ws_off; f.reg.child_s = lv.ws_off + N * 4 * mat; f.reg.child_mat = mat;
                f.reg.child_ld = int32_t(ldw);
                const int64_t N2 = N * 7;
                f.reg.grand_t = lv2.ws_off; f.reg.grand_s = lv2.ws_off + N2 * 4 * lv2.mat_words;
                f.reg.grand_q = lv2.ws_off + N2 * 8 * lv2.mat_words; f.reg.grand_mat = lv2.mat_words;
                f.reg.grand_ld = int32_t(lv2.ldw);
                if (group == 2 && odd_pair) {
                    // children of odd size: their sums are written in full (their own peeling reads them), their last
                    // row and column come from thin products, everything else as in the even pair
                    f.kind = OP_FORM2_ODD;
                    f.vec_ok = 0;
                    p->launches.push_back(f);
                    build(level + 2, gtab, N2 * 7, ctab + 1);
                    Launch x{};
                    x.kind = OP_PEEL; x.level = level + 1; x.j = -1; x.vec_ok = 0; x.peel_fused = 1;
                    x.parent_tab = ctab; x.child_tab = -1; x.count = N2; x.m = lv2.m; x.h = lv2.h;
                    x.sibling_tab = tab + 1;
                    p->launches.push_back(x);
                    Launch r = f;
                    r.kind = OP_RECOMBINE2_ODD;
                    r.peel_fused = lv.peel;
                    p->launches.push_back(r);
                } else if (group == 2) {
                    f.kind = OP_FORM2;
                    f.vec_ok = parents_even && (lv2.h & 1) == 0;
                    p->launches.push_back(f);
                    build(level + 2, gtab, N2 * 7);      // no sibling sets: the pass leaves A21 and B12 of the children's sums unwritten
                    Launch r = f;
                    r.kind = OP_RECOMBINE2;
                    r.peel_fused = lv.peel;
                    r.vec_ok = recombine_even && (lv2.h & 1) == 0;
                    p->launches.push_back(r);
                } else {
                    const LevelInfo &lv3 = p->levels[level + 2];
                    const int64_t N3 = N2 * 7;
                    const int64_t ggtab = append(bfs_children(gtab, N3, lv3));
                    if (ggtab < 0) return;
                    f.kind = OP_FORM3;
                    f.vec_ok = 0;
                    f.reg3.great_t = lv3.ws_off; f.reg3.great_s = lv3.ws_off + N3 * 4 * lv3.mat_words;
                    f.reg3.great_q = lv3.ws_off + N3 * 8 * lv3.mat_words; f.reg3.great_mat = lv3.mat_words;
                    f.reg3.great_ld = int32_t(lv3.ldw);
                    p->launches.push_back(f);
                    build(level + 3, ggtab, N3 * 7);
                    Launch r = f;
                    r.kind = OP_RECOMBINE3;
                    r.peel_fused = lv.peel;
                    p->launches.push_back(r);
                }
            } else {
                p->launches.push_back(f);
                build(level + 1, ctab, N * 7, tab + 1);
                Launch r = f;
                r.kind = OP_RECOMBINE;
                r.peel_fused = lv.peel;
                r.vec_ok = recombine_even;
                p->launches.push_back(r);
            }
        } else {
            const int64_t t_base = lv.ws_off, s_base = lv.ws_off + N * mat, q_base = lv.ws_off + 2 * N * mat;
            // Sub-problems in an order that lets each sum grow out of the one before it in the same slot:
            // T2 -> T3 = T2 - A11 -> T5 = A12 - T3, S2 -> S3 = B22 - S2 -> S6 = S3 - B21, then T4, S4 from the quadrants
            // (24 h^2 words instead of 30; same operations as Appendix A's chain).  Q0 stays first: its fold writes C.
            static constexpr int kOrder[7] = {0, 1, 2, 3, 5, 6, 4};
            for (int step = 0; step < 7; ++step) {
                const int j = kOrder[step];
                std::vector<Node> kids(static_cast<size_t>(N), Node{});
                for (int64_t q = 0; q < N; ++q) {
                    const Node nd = p->nodes[tab + q];
                    Node &k = kids[size_t(q)];
                    k.a = kTQuad[j] >= 0 ? quadrant(nd.a, kTQuad[j], h) : ws_mat(t_base + q * mat, ldw);
                    k.b = kSQuad[j] >= 0 ? quadrant(nd.b, kSQuad[j], h) : ws_mat(s_base + q * mat, ldw);
                    k.c = ws_mat(q_base + q * mat, ldw);
                }
                const int64_t ctab = append(kids);
                if (ctab < 0) return;
                Launch f{};
                f.kind = OP_FORM_ONE; f.level = level; f.j = j; f.vec_ok = parents_even;
                f.parent_tab = tab; f.child_tab = ctab; f.count = N; f.m = lv.m; f.h = h;
                f.chain = (j == 3 || j == 5 || j == 6);
               
                if (kTQuad[j] < 0 || kSQuad[j] < 0) p->launches.push_back(f);   // j = 0, 1 need no sums
                build(level + 1, ctab, N);
                if (!err.empty()) return;
                // Where the sub-problem ends in a one-level recombination pass (even size), that pass folds the product
                // into this level's C quadrants itself: Q_j is neither written nor read back.  (The two- and three-level
                // passes run one CTA per SM and cannot keep such read-modify-writes in flight beside their own loads:
                // measured slower than a fold pass of its own, so they write Q_j as before.)
                Launch &last = p->launches.back();
                const bool folds = !p->no_dfs_fold && (h & 1) == 0 &&
                                   last.kind == OP_RECOMBINE &&
                                   last.level == level + 1 && last.parent_tab == ctab;
                if (folds) {
                    last.fold = j + 1;
                    last.fold_peel = lv.peel && j == 0;
                    last.fold_tab = tab;
                    last.fold_tolerant = !recombine_even;      // the sub-problems' own matrices decide last.vec_ok
                    continue;
                }
                Launch a = f;
                a.kind = OP_ACCUMULATE;
                a.chain = 0;
                a.peel_fused = lv.peel && j == 0;
                p->launches.push_back(a);
            }
        }
        if (lv.peel) {
            Launch x{};
            x.kind = OP_PEEL; x.level = level; x.j = -1; x.vec_ok = 0; x.peel_fused = 1;
            x.parent_tab = tab; x.child_tab = -1; x.count = N; x.m = lv.m; x.h = h;
            x.sibling_tab = siblings;
            p->launches.push_back(x);
        }
    }
};

}  // namespace

// A run of BFS levels whose lower members are not peeled (their fix-ups need the children's own
// products) is cut into groups of the largest allowed size from the bottom, where the bytes are;
// what is left over forms the group at the top of the run.
int fused_group_size(const std::vector<int64_t> &sizes, const std::string &sched, int level, int max_fused, bool *odd_pair)
{
    const int L = int(sched.size());
    if (odd_pair) *odd_pair = false;
    if (max_fused <= 1 || level >= L || sched[level] != 'B') return 1;
    int run = 0;
    while (level + run < L && sched[level + run] == 'B' && (run == 0 || (sizes[level + run] & 1) == 0)) ++run;
    // A BFS level of odd size right below the run cannot be a lower member of an ordinary group, but it can be the
    // lower member of a pair (the two-level kernels for odd children): the run's last level pairs with it, and the
    // levels above are grouped among themselves.  The bytes are at the bottom, so the pair is worth more there.
    const int next = level + run;
    if (next < L && sched[next] == 'B' && (sizes[next] & 1)) {
        if (run == 1) {
            if (odd_pair) *odd_pair = true;
            return 2;
        }
        run -= 1;
    }
    if (run <= 1) return 1;
    return run % max_fused == 0 ? max_fused : run % max_fused;
}

bool fused_step_chosen(int mode, const std::string &sched, int64_t h, int64_t parents)
{
    if (sched.empty() || sched.back() != 'B' || mode == 2 || h < 1) return false;
    return mode == 1 || fused_step_pays(h, parents, kNominalSMs);
}

// What one product costs, from the quantities the kernels are bound by (measured on B200): the base products at
// the DMMA rate of their tiling, everything else as HBM bytes, a few microseconds per launch.
ModelParts plan_model_parts(const std::vector<int64_t> &sizes, const std::string &sched, int64_t batch, int fused_mode)
{
    const int L = int(sched.size());
    ModelParts out{};
    double visits = double(batch), sequential = 1.0;   // node visits at the current level; sub-trees run one after another
    const bool fused = L > 0 && fused_step_chosen(fused_mode, sched, sizes[L], [&] {
        int64_t live = batch;
        for (int i = 0; i + 1 < L; ++i)
            if (sched[i] == 'B') live *= 7;
        return live;
    }());
    const std::string upper = fused ? sched.substr(0, size_t(L) - 1) : sched;    // levels handled by streaming passes
    const int LU = int(upper.size());
    bool sibling_leaves = false;      // the nodes of the level at hand are whole sets of children of parents that are in memory in full
    for (int level = 0; level < L;) {
        const double m = double(sizes[level]), h = double(sizes[level + 1]);
        if (sizes[level] & 1) {
            // last column and last row: each reads one operand in full, or the parent's four quadrants for seven siblings
            out.pass_bytes += visits * 2.0 * m * m * 8.0 * (sibling_leaves ? 4.0 / 7.0 : 1.0);
            out.launches += 2.0 * sequential;
        }
        if (level >= LU) break;                                // the fused deepest step: accounted with the products
        if (sched[level] == 'D') {
            // 24 h^2 to form the operands one at a time (each sum grows out of the one before it); the products are folded
            // into C by the recombination pass below (24 h^2 instead of that pass's h^2 of writes) or, where the
            // sub-problem does not end in one, written and folded by a pass of their own (31 h^2)
            const bool folds = level + 1 < LU && upper[level + 1] == 'B' && (sizes[level + 1] & 1) == 0 &&
                               fused_group_size(sizes, upper, level + 1, 3, nullptr) == 1;
            out.pass_bytes += visits * (24.0 + (folds ? 23.0 : 31.0)) * h * h * 8.0;
            out.launches += (folds ? 5.0 : 12.0) * sequential;
            visits *= 7.0;
            sequential *= 7.0;
            ++level;
            sibling_leaves = false;
            continue;
        }
        bool odd_pair = false;
        const int g = fused_group_size(sizes, upper, level, 3, &odd_pair);
        sibling_leaves = g == 1 || odd_pair;
        // per parent, in h^2 of its children (a pair with odd children writes all four quadrants of their sums)
        const double words = g == 1 ? 27.0 : g == 2 ? (odd_pair ? 30.0 : 28.0) + 16.25 : 49.0 + 25.5;
        if (odd_pair) {     // the children's own last column and row: thin products over their operands
            out.pass_bytes += visits * 4.0 * 2.0 * h * h * 8.0;     // seven siblings from their parent's four quadrants
            out.launches += 2.0 * sequential;
        }
        out.pass_bytes += visits * words * h * h * 8.0;
        out.launches += 2.0 * sequential;
        for (int i = 0; i < g; ++i) visits *= 7.0;
        level += g;
    }
    if (fused) {
        // one kernel for the whole deepest step: tiles of 16 x 32 positions, h / 16 slabs each; 0.72 us per slab for a
        // CTA alone on its SM (two warps per tile), 1.25 us when two share one (measured at h = 256, 384, 512)
        const double h = double(sizes[L]);
        const double tiles = double((sizes[L] + 15) / 16) * double((sizes[L] + 31) / 32) * visits / sequential;
        const double slabs = double((sizes[L] + 15) / 16);
        const double per_launch = tiles <= kNominalSMs ? slabs * 0.72 : double(int64_t((tiles + 2 * kNominalSMs - 1) / (2 * kNominalSMs))) * slabs * 1.25;
        out.product_us += per_launch * sequential;
        out.product_flops += visits * 7.0 * 2.0 * h * h * h;
        // launched as a programmatic dependent: its launch and ramp-up run under the tail of the kernel before it
        out.launches += sequential / 3.0;
        return out;
    }
    const int64_t b = sizes[L];
    const double leaves = visits, kp = double((b + 15) / 16 * 16);
    const int rem = gemm_thin_remainder(b);
    out.product_flops = leaves * 2.0 * double(b) * double(b) * double(b);
    if (b - rem > 0) {
        GemmRegion regions[4];
        const int64_t count = leaves > 4.0e9 ? int64_t(4e9) : int64_t(leaves);
        const int nreg = gemm_regions(b - rem, count, kNominalSMs, regions);
        const double wide_tile_us = kp / 16.0 * 2.147 + 1.1;      // one 128 x 128 tile on an SM: per 16-deep slab and per tile
        for (int i = 0; i < nreg; ++i) {
            const GemmRegion &r = regions[i];
            const int t = r.small ? 64 : 128;
            double slots = r.small ? 2.0 * kNominalSMs : double(kNominalSMs);
            double tile_us = r.small ? wide_tile_us * 0.5 / 0.88 : wide_tile_us;
            double tiles = double((r.row_end - r.row0 + t - 1) / t) * double((r.col_end - r.col0 + t - 1) / t) * double(r.leaves);
            if (r.small && gemm_uses_tiny_tiles(int64_t(tiles / sequential), kNominalSMs)) {
                // 32 x 64 tiles: twice as many, a fifth of a large tile's time each while an SM holds one or two of them
                tiles *= 2.0;
                slots = 1.5 * kNominalSMs;
                tile_us = wide_tile_us * 0.2;
            }
            double rounds = tiles / sequential / slots;          // per launch: a DFS level above runs its sub-trees one by one
            if (rounds < 1.0) rounds = 1.0;
            out.product_us += rounds * tile_us * sequential;
            out.launches += sequential;
        }
    }
    if (rem) {
        // one operand of every leaf read in full for each of the two strips, or the four quadrants of the parent for seven leaves
        out.thin_bytes += leaves * 2.0 * double(b) * double(b) * 8.0 * (sibling_leaves && b > 64 ? 4.0 / 7.0 : 1.0);
        out.launches += 2.0 * sequential;
    }
    return out;
}

// Only used to decide which candidates are tried first and to pick plans created with cutoff 0; the autotuner's
// choice itself is by measurement.
double plan_model_ms(const std::vector<int64_t> &sizes, const std::string &sched, int64_t batch, int fused_mode)
{
    const double hbm = 6.2e12, launch_us = 3.0;
    const ModelParts m = plan_model_parts(sizes, sched, batch, fused_mode);
    return m.product_us * 1e-3 + (m.pass_bytes + m.thin_bytes) / hbm * 1e3 + m.launches * launch_us * 1e-3;
}


bool model_choice(int64_t n, int64_t batch, int64_t budget_words, int64_t min_base, int fused_mode,
                  std::vector<int64_t> *sizes_out, std::string *sched_out)
{
    std::vector<int64_t> chain{n};
    while (chain.back() / 2 >= min_base && chain.size() <= 10) chain.push_back(chain.back() / 2);
    double best = -1.0;
    for (size_t L = 0; L < chain.size(); ++L) {
        const std::vector<int64_t> sizes(chain.begin(), chain.begin() + L + 1);
        for (unsigned mask = 0; mask < (1u << L); ++mask) {
            std::string sched(L, 'B');
            for (size_t i = 0; i < L; ++i)
                if (mask >> i & 1) sched[i] = 'D';
            const int64_t words = actual_workspace_words(sizes, sched, batch);
            if (words < 0 || words > budget_words) continue;
            double nodes = double(batch), level_nodes = double(batch);      // entries the node tables would need
            for (size_t i = 0; i < L; ++i) nodes += (level_nodes *= 7.0);
            if (nodes > double(kMaxNodes)) continue;
            const double ms = plan_model_ms(sizes, sched, batch, fused_mode);
            if (best < 0 || ms < best) {
                best = ms;
                *sizes_out = sizes;
                *sched_out = sched;
            }
        }
    }
    return best >= 0;
}

std::vector<int64_t> level_sizes(int64_t n, int64_t cutoff)
{
    std::vector<int64_t> m{n};
    while (m.back() > cutoff) m.push_back(m.back() / 2);
    return m;
}

int64_t actual_workspace_words(const std::vector<int64_t> &sizes, const std::string &sched, int64_t batch)
{
    if (!sched_ok(sizes, sched)) return -1;
    int64_t words = 0, live = batch;
    for (size_t i = 0; i < sched.size(); ++i) {
        const int64_t h = sizes[i + 1];
        const int64_t mat = round_up(h * round_up(h, 4), kPadWords);
        const int64_t per_parent = sched[i] == 'B' ? 15 : 3;
        if (live > std::numeric_limits<int64_t>::max() / (per_parent * mat) - 1) return std::numeric_limits<int64_t>::max() / 16;
        words += live * per_parent * mat;
        if (words < 0 || words > std::numeric_limits<int64_t>::max() / 16) return std::numeric_limits<int64_t>::max() / 16;
        if (sched[i] == 'B') live *= 7;
    }
    return words;
}

int64_t model_workspace_words(const std::vector<int64_t> &sizes, const std::string &sched, int64_t batch,
                              int accounting)
{
    if (!sched_ok(sizes, sched) || (accounting != 15 && accounting != 21)) return -1;
    long double words = 0;
    int64_t live = batch;
    for (size_t i = 0; i < sched.size(); ++i) {
        const long double h = (long double)sizes[i + 1];
        words += (long double)live * (sched[i] == 'B' ? accounting : 3) * h * h;
        if (sched[i] == 'B') live *= 7;
    }
    if (words > 1.0e18L) return std::numeric_limits<int64_t>::max() / 16;
    return int64_t(words);
}

bool lm_schedule(const std::vector<int64_t> &sizes, int64_t batch, int64_t budget_words, std::string *out)
{
    const size_t L = sizes.size() - 1;
    for (size_t ell = 0; ell <= L; ++ell) {
        std::string s = std::string(ell, 'D') + std::string(L - ell, 'B');
        const int64_t w = actual_workspace_words(sizes, s, batch);
        if (w >= 0 && w <= budget_words) {
            *out = s;
            return true;
        }
    }
    return false;
}

std::string build_plan(PlanDesc *p)
{
    if (!sched_ok(p->sizes, p->schedule)) return "schedule does not match the number of levels";
    const int L = int(p->sizes.size()) - 1;
    p->levels.clear();
    p->nodes.clear();
    p->launches.clear();
    int64_t live = p->batch, off = 0;
    for (int i = 0; i < L; ++i) {
        LevelInfo lv{};
        lv.m = p->sizes[i];
        lv.h = p->sizes[i + 1];
        lv.ldw = round_up(lv.h, 4);
        lv.mat_words = round_up(lv.h * lv.ldw, kPadWords);
        lv.parents = live;
        lv.ws_off = off;
        lv.mode = p->schedule[i];
        lv.peel = (lv.m & 1) != 0;
        off += live * (lv.mode == 'B' ? 15 : 3) * lv.mat_words;
        if (lv.mode == 'B') live *= 7;
        if (live > kMaxNodes) return "recursion tree too large for the node tables (more than 2^23 nodes)";
        p->levels.push_back(lv);
    }
    const bool scaling = p->scale_inside || p->scale_outside;
    if (scaling) {
        // scaled copies of A and B (packed rows) and three int32 exponent vectors per batch member
        p->scale_ld = round_up(p->n, 4);
        const int64_t copy_words = round_up(p->batch * p->n * p->scale_ld, kPadWords);
        p->scale_a_off = off;
        p->scale_b_off = off + copy_words;
        p->scale_exp_off = off + 2 * copy_words;
        off = p->scale_exp_off + round_up((3 * p->batch * p->n + 1) / 2, kPadWords);
    }
    p->ws_words = off;

    std::vector<Node> top(static_cast<size_t>(p->batch), Node{});
    for (int64_t b = 0; b < p->batch; ++b) {
        if (scaling) {
            top[size_t(b)].a = ws_mat(p->scale_a_off + b * p->n * p->scale_ld, p->scale_ld);
            top[size_t(b)].b = ws_mat(p->scale_b_off + b * p->n * p->scale_ld, p->scale_ld);
        } else {
            top[size_t(b)].a = Operand{b * p->stride_a, int32_t(p->lda), BASE_A};
            top[size_t(b)].b = Operand{b * p->stride_b, int32_t(p->ldb), BASE_B};
        }
        top[size_t(b)].c = Operand{b * p->stride_c, int32_t(p->ldc), BASE_C};
    }
    Builder bld{p, {}};
    const int64_t tab = bld.append(top);
    if (tab < 0) return bld.err;
    if (scaling) {
        Launch in{};
        in.kind = OP_SCALE_IN; in.count = p->batch; in.m = p->n;
        p->launches.push_back(in);
    }
    bld.build(0, tab, p->batch);
    if (scaling && bld.err.empty()) {
        Launch out{};
        out.kind = OP_SCALE_OUT; out.count = p->batch; out.m = p->n;
        p->launches.push_back(out);
    }
    return bld.err;
}

}  // namespace strassen
