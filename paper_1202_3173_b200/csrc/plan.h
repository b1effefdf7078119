// Internal host-side description of one planned product: level sizes, the resolved
// BFS/DFS schedule, the workspace carve-up, the node tables and the launch list that
// strassen_dgemm replays.  Nothing here touches the device.
#pragma once
#include <cstddef>
#include <cstdint>
#include <string>
#include <vector>

namespace strassen {

// Which allocation an operand lives in.  User pointers arrive per call, so the node
// tables store (base id, element offset, leading dimension) and the kernels resolve
// addresses from the four base pointers they get as arguments.
enum Base : int32_t { BASE_A = 0, BASE_B = 1, BASE_C = 2, BASE_WS = 3 };

struct Operand {
    int64_t off;   // element offset from the base pointer
    int32_t ld;    // leading dimension in elements
    int32_t base;  // Base
};

// One live node of the recursion tree: its two factors and where its product goes.
struct Node {
    Operand a, b, c;
};
static_assert(sizeof(Node) == 48, "Node is copied to the device as is");

enum OpKind : int32_t {
    OP_FORM = 0,       // BFS: T2..T5, S2,S3,S4,S6 of `count` parents -> 7*count children
    OP_GEMM = 1,       // base products of `count` leaves of size m
    OP_RECOMBINE = 2,  // BFS: 7 Q of each parent -> its four C quadrants
    OP_FORM_ONE = 3,   // DFS: operands of child j of each parent
    OP_ACCUMULATE = 4, // DFS: fold Q_j of each parent into its C quadrants
    OP_PEEL = 5,       // odd m: rank-one update, last column, last row
    OP_FORM2 = 6,      // two BFS levels at once: sums of the children and of the grandchildren
    OP_RECOMBINE2 = 7, // two BFS levels at once: 49 grandchild products -> the parent's C
    OP_SCALE_IN = 8,   // diagonal scaling: exponents, scaled copies of A and B in the workspace
    OP_SCALE_OUT = 9,  // diagonal scaling: C scaled back in place
    OP_FORM3 = 10,     // three BFS levels at once: sums of the children, grandchildren and great-grandchildren
    OP_RECOMBINE3 = 11, // three BFS levels at once: 343 great-grandchild products -> the parent's C
    OP_FUSED_STEP = 12, // a whole BFS step of the deepest level in one kernel: quadrants of A, B -> C
    OP_FORM2_ODD = 14,      // two BFS levels at once where the children have odd size (peeled)
    OP_RECOMBINE2_ODD = 15, // ... and their recombination
    OP_LINCOMB = 13     // generic bilinear scheme: one output matrix per parent as a linear combination (j = index of its LinComb)
};

// Regular layout of the workspace regions a two- or three-level launch writes / reads (element offsets
// from the workspace base; slot s of child c sits at base + (c * slots + s) * mat).
struct Regions2 {
    int64_t child_t, child_s;            // level i+1 operand sums: 4 per parent and side
    int64_t child_mat;
    int64_t grand_t, grand_s, grand_q;   // level i+2: 4 + 4 sums and 7 products per child
    int64_t grand_mat;
    int32_t child_ld, grand_ld;
};

// The third level of a three-level launch, laid out like the second.
struct Regions3 {
    int64_t great_t, great_s, great_q;   // level i+3: 4 + 4 sums and 7 products per grandchild
    int64_t great_mat;
    int32_t great_ld;
};

struct Launch {
    int32_t kind;        // OpKind
    int32_t level;       // recursion level of the parents (of the leaves for OP_GEMM)
    int32_t j;           // sub-problem index for OP_FORM_ONE / OP_ACCUMULATE
    int32_t vec_ok;      // every operand offset and ld involved is even (16-byte accesses
                         // are legal provided the base pointers are 16-byte aligned)
    int64_t parent_tab;  // index of the first parent (leaf) node in the table
    int64_t child_tab;   // index of the first child node (unused for OP_GEMM / OP_PEEL)
    int64_t count;       // number of parents (leaves)
    int64_t m;           // size of the parents (leaves)
    int64_t h;           // size of the children
    int32_t peel_fused;  // recombine / accumulate(j = 0) of an odd-size parent: also add the rank-one term
                         // A[:, m-1] x B[m-1, :] of the peeled split; on OP_PEEL: that term is already in C
    int64_t grand_tab;   // OP_FORM2 / OP_RECOMBINE2: index of the first grandchild node
    int32_t chain;       // OP_FORM_ONE: the operand is formed from the previous content of its slot (T3 from T2, T5 from T3,
                         // S3 from S2, S6 from S3) instead of from the quadrants alone
    int32_t fold;        // OP_RECOMBINE / 2 / 3 whose parents are the sub-problems j of a DFS step one level up: 1 + j, and their
                         // products are folded straight into the DFS parents' C quadrants instead of being written (0: no fold)
    int32_t fold_peel;   // ... and the DFS parents have odd size: the first fold (j = 0) carries their rank-one term
    int64_t fold_tab;    // ... index of the first DFS parent node (DFS parent i owns sub-problem node i)
    int32_t fold_tolerant;   // ... whose C (or B, for the rank-one term) does not allow the 16-byte accesses the sub-problems' own
                             // matrices allow: the fold checks the alignment of every access to them
    int64_t sibling_tab; // OP_GEMM / OP_PEEL whose nodes are the complete sets of seven children of the nodes of a BFS step, child j
                         // of parent i at node 7 i + j, and those parents' operands are in memory in full (the even multi-level
                         // passes skip one quadrant of the intermediate sums): 1 + index of the first of those parents
                         // (0: none); lets the thin products of all seven be computed from the parents' quadrants
    Regions2 reg;        // OP_FORM2 / OP_RECOMBINE2 / OP_FORM3 / OP_RECOMBINE3 only
    Regions3 reg3;       // OP_FORM3 / OP_RECOMBINE3 only
};

struct LevelInfo {
    int64_t m;          // size of a node at this level
    int64_t h;          // size of its children, floor(m / 2)
    int64_t ldw;        // leading dimension of the children's workspace matrices
    int64_t mat_words;  // padded words of one such matrix
    int64_t parents;    // live nodes at this level (batch * 7^{#B above})
    int64_t ws_off;     // first word of this level's workspace region
    char mode;          // 'B' or 'D'
    bool peel;          // m odd
};

struct PlanDesc {
    int64_t n = 0, cutoff = 0, batch = 1;
    int64_t lda = 0, ldb = 0, ldc = 0;
    int64_t stride_a = 0, stride_b = 0, stride_c = 0;
    int max_fused_levels = 3;       // consecutive BFS levels formed / recombined by one pass: up to 3, 2 or 1
    bool no_dfs_fold = false;       // keep the separate fold pass of a DFS step even where the pass below could fold
    int fused_step = 0;             // deepest BFS step as one kernel: 0 = where the rule says it pays, 1 = always, 2 = never
    bool scale_inside = false, scale_outside = false;   // diagonal scaling (Section 6.1)
    int64_t scale_a_off = 0, scale_b_off = 0, scale_exp_off = 0, scale_ld = 0;   // workspace words / leading dimension
    std::string schedule;           // resolved, one char per level
    std::vector<int64_t> sizes;     // m_0 .. m_L
    std::vector<LevelInfo> levels;  // L entries
    int64_t ws_words = 0;           // total workspace words
    std::vector<Node> nodes;        // all node tables, concatenated
    std::vector<Launch> launches;   // replayed in order by strassen_dgemm
    std::vector<unsigned char> lincombs;   // generic bilinear schemes: the LinComb records OP_LINCOMB launches refer to (bilinear.h)
    int scheme_n0 = 0, scheme_q = 0;       // ... and the scheme's shape (0: the Strassen-Winograd plan of Appendix A)
};

// How many levels, starting at `level`, one pass forms and recombines (1 .. max_fused) under schedule
// `sched` with level sizes `sizes`; 1 for a DFS level.
int fused_group_size(const std::vector<int64_t> &sizes, const std::string &sched, int level, int max_fused,
                     bool *odd_pair = nullptr);   // *odd_pair: a pair whose lower member has odd size

// Whether the deepest level (a BFS step over `parents` nodes with children of size h) runs as one fused kernel.
bool fused_step_chosen(int mode, const std::string &sched, int64_t h, int64_t parents);

// Cost-model estimate (milliseconds on a B200) of one product with level sizes `sizes` (m_0 .. m_L) and
// schedule `sched`; orders the autotuner's search and picks plans created with cutoff 0.
double plan_model_ms(const std::vector<int64_t> &sizes, const std::string &sched, int64_t batch, int fused_mode = 0);

// The parts of that estimate, also reported as the plan's algorithmic work: bytes the streaming passes move as
// scheduled (multi-level passes counted with what they really read and write; DFS steps with their surcharge;
// peeled columns and rows), bytes of the thin remainder products, time and flops of the base products, launches.
struct ModelParts {
    double pass_bytes, thin_bytes, product_us, product_flops, launches;
};
ModelParts plan_model_parts(const std::vector<int64_t> &sizes, const std::string &sched, int64_t batch, int fused_mode = 0);

// The (level sizes, schedule) of least estimated time among all step counts whose base size is >= min_base
// and all B/D strings whose workspace fits budget_words.  False if nothing fits (cannot happen: zero levels
// need no workspace).
bool model_choice(int64_t n, int64_t batch, int64_t budget_words, int64_t min_base, int fused_mode,
                  std::vector<int64_t> *sizes_out, std::string *sched_out);

// Level sizes m_0 = n, m_{i+1} = floor(m_i / 2) while m_i > cutoff.
std::vector<int64_t> level_sizes(int64_t n, int64_t cutoff);

// Words of workspace the library itself needs for a schedule (quadrant operands used in
// place, padded rows); 0 levels -> 0.  Returns -1 if the schedule is malformed.
int64_t actual_workspace_words(const std::vector<int64_t> &sizes, const std::string &sched, int64_t batch);

// Words under the paper's accounting (21 quarter matrices per BFS parent, 3 per DFS parent)
// or the 15-matrix variant; unpadded.  Returns -1 if the schedule is malformed.
int64_t model_workspace_words(const std::vector<int64_t> &sizes, const std::string &sched, int64_t batch,
                              int accounting);

// Limited-Memory rule: fewest leading 'D', then 'B' only, that fits budget_words.
// Returns false if even all-'D' does not fit.
bool lm_schedule(const std::vector<int64_t> &sizes, int64_t batch, int64_t budget_words, std::string *out);

// Fill levels, workspace layout, node tables and launch list from the scalar fields,
// sizes and schedule already set in `p`.  Returns an empty string or an error text.
std::string build_plan(PlanDesc *p);

}  // namespace strassen
