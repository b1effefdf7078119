// Streaming kernels of one Strassen-Winograd step (Appendix A): operand formation,
// recombination, the one-sub-problem-at-a-time variants of a DFS step (Algorithm 1) and the
// peeling fix-ups for odd sizes.  All are HBM-bound: every element of every quadrant is read
// once and every output element written once per level.
//
// Work decomposition shared by the four add kernels: a CTA of 64 x 4 threads owns a tile of
// 16 rows x (64 * VEC) columns of one h x h quadrant position of one (node, side) item;
// each thread handles 4 rows (stride 4) and VEC adjacent columns, issuing all of its loads
// before the arithmetic so that 4 x (number of input streams) requests are in flight.
#include "kernels.h"
#include "fold.cuh"

namespace strassen {

namespace {

constexpr int TX = 64, TY = 4, ROWS_PER_THREAD = 4, TILE_ROWS = TY * ROWS_PER_THREAD;
constexpr int MAX_Z = kMaxItemsPerLaunch;   // items per launch (gridDim.z limit is 65535)

// ---------------------------------------------------------------------------------------
// BFS operand formation.  item = 2 * parent + side; side 0 forms T2..T5 from the quadrants
// of the parent's A operand, side 1 forms S2, S3, S4, S6 from those of its B operand:
//   T2 = A21 + A22   T3 = T2 - A11   T4 = A11 - A21   T5 = A12 - T3
//   S2 = B12 - B11   S3 = B22 - S2   S4 = B22 - B12   S6 = S3 - B21
// ---------------------------------------------------------------------------------------
template <int VEC, int RPT>
__global__ void __launch_bounds__(TX *TY) form_bfs_kernel(const Node *__restrict__ parents,
                                                          const Node *__restrict__ children, Bases bases, int h,
                                                          int item0)
{
    using V = Vec<VEC>;
    using T = typename V::type;
    const int item = item0 + blockIdx.z;
    const int par = item >> 1, side = item & 1;
    const int c = (blockIdx.x * TX + threadIdx.x) * VEC;
    if (c >= h) return;
    const Node *kids = children + size_t(par) * 7;
    const Operand x = side ? parents[par].b : parents[par].a;
    const double *X = resolve(bases, x);
    const int64_t ld = x.ld;
    const int64_t hq = int64_t(h) * ld;
    double *o0, *o1, *o2, *o3;
    int64_t ldo;
    if (side == 0) {
        o0 = resolve(bases, kids[2].a); o1 = resolve(bases, kids[3].a);
        o2 = resolve(bases, kids[4].a); o3 = resolve(bases, kids[5].a);
        ldo = kids[2].a.ld;
    } else {
        o0 = resolve(bases, kids[2].b); o1 = resolve(bases, kids[3].b);
        o2 = resolve(bases, kids[4].b); o3 = resolve(bases, kids[6].b);
        ldo = kids[2].b.ld;
    }
    const int r0 = blockIdx.y * (TY * RPT) + threadIdx.y;
    T x11[RPT], x12[RPT], x21[RPT], x22[RPT];
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
        const int r = r0 + i * TY;
        if (r < h) {
            const double *q = X + int64_t(r) * ld + c;
            x11[i] = V::ld(q); x12[i] = V::ld(q + h); x21[i] = V::ld(q + hq); x22[i] = V::ld(q + hq + h);
        }
    }
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
        const int r = r0 + i * TY;
        if (r < h) {
            const int64_t o = int64_t(r) * ldo + c;
            if (side == 0) {
                const T t2 = V::add(x21[i], x22[i]);
                const T t3 = V::sub(t2, x11[i]);
                V::st(o0 + o, t2); V::st(o1 + o, t3);
                V::st(o2 + o, V::sub(x11[i], x21[i]));
                V::st(o3 + o, V::sub(x12[i], t3));
            } else {
                const T s2 = V::sub(x12[i], x11[i]);
                const T s3 = V::sub(x22[i], s2);
                V::st(o0 + o, s2); V::st(o1 + o, s3);
                V::st(o2 + o, V::sub(x22[i], x12[i]));
                V::st(o3 + o, V::sub(s3, x21[i]));
            }
        }
    }
}

// ---------------------------------------------------------------------------------------
// BFS recombination.  item = parent:
//   U1 = Q0 + Q3   U2 = U1 + Q4   U3 = U1 + Q2
//   C11 = Q0 + Q1  C12 = U3 + Q5  C21 = U2 - Q6  C22 = U2 + Q2
// ---------------------------------------------------------------------------------------
template <int VEC, int RPT, int FOLD>      // FOLD: 0 = write the product, 1 = fold it, 2 = fold it into a parent that needs tolerant accesses
__global__ void __launch_bounds__(TX *TY) recombine_bfs_kernel(const Node *__restrict__ parents,
                                                               const Node *__restrict__ children, Bases bases,
                                                               int h, int item0, int peel, const Node *__restrict__ dfs_parents,
                                                               int fold, int fold_peel)
{
    // FOLD (fold != 0): the parents are the sub-problems j = fold - 1 of a DFS step one level up; their products are not
    // written but folded into the C quadrants of those DFS parents (size 2 * (2h)).
    // peel != 0: the parent has odd size 2h + 1; the rank-one term A[r][2h] * B[2h][c] of the peeled split
    // is added to every entry on its way out (saves a read-modify-write pass over C).
    using V = Vec<VEC>;
    using T = typename V::type;
    // last parent first: its products are the ones the preceding kernel wrote last, so they are still in L2
    const int par = item0 + (gridDim.z - 1 - blockIdx.z);
    const int c = (blockIdx.x * TX + threadIdx.x) * VEC;
    if (c >= h) return;
    const double *acol = nullptr;
    int64_t lda = 0;
    T b0 = T(), b1 = T();
    if (peel) {
        const Operand pa = parents[par].a, pb = parents[par].b;
        acol = resolve(bases, pa) + 2 * h;
        lda = pa.ld;
        const double *brow = resolve(bases, pb) + int64_t(2 * h) * pb.ld + c;
        b0 = V::ldk(brow);
        b1 = V::ldk(brow + h);
    }
    const Node *kids = children + size_t(par) * 7;
    const double *Q[7];
#pragma unroll
    for (int j = 0; j < 7; ++j) Q[j] = resolve(bases, kids[j].c);
    const int64_t ldq = kids[0].c.ld;
    const Operand cc = parents[par].c;
    double *C = resolve(bases, cc);
    const int64_t ldc = cc.ld, hq = int64_t(h) * ldc;
    FoldTarget ft{};
    if (FOLD) ft = fold_target(dfs_parents[par], bases, 2 * h, fold - 1, fold_peel);
    const int r0 = blockIdx.y * (TY * RPT) + threadIdx.y;
    constexpr int RP = RPT < 2 ? RPT : 2;   // rows per pass: 14 vectors in flight per thread
#pragma unroll
    for (int pass = 0; pass < RPT / RP; ++pass) {
        T q[RP][7];
#pragma unroll
        for (int i = 0; i < RP; ++i) {
            const int r = r0 + (pass * RP + i) * TY;
            if (r < h) {
#pragma unroll
                for (int j = 0; j < 7; ++j) q[i][j] = V::ld(Q[j] + int64_t(r) * ldq + c);
            }
        }
#pragma unroll
        for (int i = 0; i < RP; ++i) {
            const int r = r0 + (pass * RP + i) * TY;
            if (r < h) {
                const T u1 = V::add(q[i][0], q[i][3]);
                const T u2 = V::add(u1, q[i][4]);
                const T u3 = V::add(u1, q[i][2]);
                double *o = C + int64_t(r) * ldc + c;
                T c11 = V::add(q[i][0], q[i][1]), c12 = V::add(u3, q[i][5]);
                T c21 = V::sub(u2, q[i][6]), c22 = V::add(u2, q[i][2]);
                if (peel) {
                    const double a0 = acol[int64_t(r) * lda], a1 = acol[int64_t(r + h) * lda];
                    c11 = V::fma1(a0, b0, c11); c12 = V::fma1(a0, b1, c12);
                    c21 = V::fma1(a1, b0, c21); c22 = V::fma1(a1, b1, c22);
                }
                if (FOLD) {
                    fold_emit<VEC, FOLD == 2>(ft, r, c, c11);
                    fold_emit<VEC, FOLD == 2>(ft, r, c + h, c12);
                    fold_emit<VEC, FOLD == 2>(ft, r + h, c, c21);
                    fold_emit<VEC, FOLD == 2>(ft, r + h, c + h, c22);
                } else {
                    V::st(o, c11);
                    V::st(o + h, c12);
                    V::st(o + hq, c21);
                    V::st(o + hq + h, c22);
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------
// DFS operand formation of sub-problem j (Algorithm 1: "locally compute S_i and T_i").
// sides: bit 0 = the A-side operand of child j is a sum, bit 1 = the B-side one is.
// ---------------------------------------------------------------------------------------
template <int VEC>
__global__ void __launch_bounds__(TX *TY) form_one_kernel(const Node *__restrict__ parents,
                                                          const Node *__restrict__ children, Bases bases, int h,
                                                          int j, int sides, int item0, int chain)
{
    // chain != 0: the slot still holds the sum formed for the sub-problem before this one, and the new sum grows out
    // of it in place: T3 = T2 - A11, T5 = A12 - T3, S3 = B22 - S2, S6 = S3 - B21 (Appendix A's own chain).
    using V = Vec<VEC>;
    using T = typename V::type;
    const int item = item0 + blockIdx.z;
    int par, side;
    if (sides == 3) { par = item >> 1; side = item & 1; }
    else { par = item; side = sides == 2; }
    const int c = (blockIdx.x * TX + threadIdx.x) * VEC;
    if (c >= h) return;
    const Operand x = side ? parents[par].b : parents[par].a;
    const Operand y = side ? children[par].b : children[par].a;
    const double *X = resolve(bases, x);
    double *O = resolve(bases, y);
    const int64_t ld = x.ld, hq = int64_t(h) * ld, ldo = y.ld;
    const int r0 = blockIdx.y * TILE_ROWS + threadIdx.y;
    const int which = side * 8 + j + (chain ? 16 : 0);
#pragma unroll
    for (int i = 0; i < ROWS_PER_THREAD; ++i) {
        const int r = r0 + i * TY;
        if (r >= h) continue;
        const double *q = X + int64_t(r) * ld + c;
        double *slot = O + int64_t(r) * ldo + c;
        T v;
        switch (which) {
        case 16 + 3: v = V::sub(V::ldk(slot), V::ld(q)); break;                 // T3 = T2 - A11
        case 16 + 5: v = V::sub(V::ld(q + h), V::ldk(slot)); break;             // T5 = A12 - T3
        case 16 + 11: v = V::sub(V::ld(q + hq + h), V::ldk(slot)); break;       // S3 = B22 - S2
        case 16 + 14: v = V::sub(V::ldk(slot), V::ld(q + hq)); break;           // S6 = S3 - B21
        case 2: v = V::add(V::ld(q + hq), V::ld(q + hq + h)); break;                                   // T2
        case 3: v = V::sub(V::add(V::ld(q + hq), V::ld(q + hq + h)), V::ld(q)); break;                 // T3
        case 4: v = V::sub(V::ld(q), V::ld(q + hq)); break;                                            // T4
        case 5: v = V::sub(V::ld(q + h), V::sub(V::add(V::ld(q + hq), V::ld(q + hq + h)), V::ld(q))); break;  // T5
        case 10: v = V::sub(V::ld(q + h), V::ld(q)); break;                                            // S2
        case 11: v = V::sub(V::ld(q + hq + h), V::sub(V::ld(q + h), V::ld(q))); break;                 // S3
        case 12: v = V::sub(V::ld(q + hq + h), V::ld(q + h)); break;                                   // S4
        default: v = V::sub(V::sub(V::ld(q + hq + h), V::sub(V::ld(q + h), V::ld(q))), V::ld(q + hq)); break;  // S6
        }
        V::st(slot, v);
    }
}

// ---------------------------------------------------------------------------------------
// DFS fold of Q_j into C as a pass of its own, for sub-problems that do not end in a recombination
// pass (a leaf product, a DFS step or a fused step below): reads the Q_j the sub-problem wrote.
// ---------------------------------------------------------------------------------------
template <int VEC>
__global__ void __launch_bounds__(TX *TY) accumulate_kernel(const Node *__restrict__ parents,
                                                            const Node *__restrict__ children, Bases bases, int h,
                                                            int j, int item0, int peel)
{
    using V = Vec<VEC>;
    const int par = item0 + blockIdx.z;
    const int c = (blockIdx.x * TX + threadIdx.x) * VEC;
    if (c >= h) return;
    const Operand qq = children[par].c;
    const double *Q = resolve(bases, qq);
    const int64_t ldq = qq.ld;
    const FoldTarget ft = fold_target(parents[par], bases, h, j, peel);
    const int r0 = blockIdx.y * TILE_ROWS + threadIdx.y;
#pragma unroll
    for (int i = 0; i < ROWS_PER_THREAD; ++i) {
        const int r = r0 + i * TY;
        if (r >= h) continue;
        fold_emit<VEC>(ft, r, c, V::ld(Q + int64_t(r) * ldq + c));
    }
}

// ---------------------------------------------------------------------------------------
// Two BFS levels of operand formation in one pass.  A thread at (r, c) of the q x q grid
// (q = quarter of the parent's even part) reads the parent's operand X at its 16 block
// positions X[a][b] (block row a, block column b of the 4 x 4 partition), forms the four
// sums of the children at each of their four quadrant positions (u, v) -- still written,
// because the grandchildren's quadrant operands are views into them -- and from the seven
// child operands Y_j(u, v) the four sums of each child's own children.  The parent is read
// once instead of the children's operands being read back: 4 h^2 read + 10 h^2 written per
// side instead of 11 h^2 + 11 h^2.  Same operations in the same order as two single passes.
// ---------------------------------------------------------------------------------------
template <int VEC>
__global__ void __launch_bounds__(TX *TY) form2_kernel(const Node *__restrict__ parents, Bases bases, Regions2 reg,
                                                       int q, int item0)
{
    using V = Vec<VEC>;
    using T = typename V::type;
    const int item = item0 + blockIdx.z;
    const int par = item >> 1, side = item & 1;
    const int c = (blockIdx.x * TX + threadIdx.x) * VEC;
    if (c >= q) return;
    const Operand x = side ? parents[par].b : parents[par].a;
    const double *X = resolve(bases, x);
    const int64_t ld = x.ld;
    double *ws = bases.p[BASE_WS];
    double *child = ws + (side ? reg.child_s : reg.child_t) + int64_t(par) * 4 * reg.child_mat;
    double *grand = ws + (side ? reg.grand_s : reg.grand_t) + int64_t(par) * 28 * reg.grand_mat;
    const int64_t cld = reg.child_ld, gld = reg.grand_ld;
    const int r0 = blockIdx.y * TILE_ROWS + threadIdx.y;
#pragma unroll 1
    for (int i = 0; i < ROWS_PER_THREAD; ++i) {
        const int r = r0 + i * TY;
        if (r >= q) break;
        T xv[4][4];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) xv[a][b] = V::ld(X + (int64_t(a) * q + r) * ld + b * q + c);
        T y[7][2][2];   // operand of child j at quadrant position (u, v)
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int v = 0; v < 2; ++v) {
                const T x11 = xv[u][v], x12 = xv[u][2 + v], x21 = xv[2 + u][v], x22 = xv[2 + u][2 + v];
                T s0, s1, s2, s3;
                if (side == 0) {
                    s0 = V::add(x21, x22);      // T2
                    s1 = V::sub(s0, x11);       // T3
                    s2 = V::sub(x11, x21);      // T4
                    s3 = V::sub(x12, s1);       // T5
                    y[0][u][v] = x11; y[1][u][v] = x12; y[2][u][v] = s0; y[3][u][v] = s1;
                    y[4][u][v] = s2; y[5][u][v] = s3; y[6][u][v] = x22;
                } else {
                    s0 = V::sub(x12, x11);      // S2
                    s1 = V::sub(x22, s0);       // S3
                    s2 = V::sub(x22, x12);      // S4
                    s3 = V::sub(s1, x21);       // S6
                    y[0][u][v] = x11; y[1][u][v] = x21; y[2][u][v] = s0; y[3][u][v] = s1;
                    y[4][u][v] = s2; y[5][u][v] = x22; y[6][u][v] = s3;
                }
                // Below this pass the children's sums are read only as quadrant operands: X11, X12, X22 on the
                // A side, X11, X21, X22 on the B side.  The fourth block is never read and is not written.
                if (side == 0 ? !(u == 1 && v == 0) : !(u == 0 && v == 1)) {
                    const int64_t o = (int64_t(u) * q + r) * cld + v * q + c;
                    V::st(child + o, s0);
                    V::st(child + reg.child_mat + o, s1);
                    V::st(child + 2 * reg.child_mat + o, s2);
                    V::st(child + 3 * reg.child_mat + o, s3);
                }
            }
        const int64_t og = int64_t(r) * gld + c;
#pragma unroll
        for (int j = 0; j < 7; ++j) {
            const T y11 = y[j][0][0], y12 = y[j][0][1], y21 = y[j][1][0], y22 = y[j][1][1];
            double *g = grand + int64_t(j) * 4 * reg.grand_mat + og;
            if (side == 0) {
                const T t2 = V::add(y21, y22);
                const T t3 = V::sub(t2, y11);
                V::st(g, t2);
                V::st(g + reg.grand_mat, t3);
                V::st(g + 2 * reg.grand_mat, V::sub(y11, y21));
                V::st(g + 3 * reg.grand_mat, V::sub(y12, t3));
            } else {
                const T s2 = V::sub(y12, y11);
                const T s3 = V::sub(y22, s2);
                V::st(g, s2);
                V::st(g + reg.grand_mat, s3);
                V::st(g + 2 * reg.grand_mat, V::sub(y22, y12));
                V::st(g + 3 * reg.grand_mat, V::sub(s3, y21));
            }
        }
    }
}

// ---------------------------------------------------------------------------------------
// Two BFS levels of recombination in one pass: the 49 grandchild products of a parent at
// (r, c) give, child by child, that child's product at its four quadrant positions (kept in
// registers, never written), and those give the parent's C at its 16 block positions:
// 12.25 h^2 read + 4 h^2 written instead of 19.25 h^2 + 11 h^2.
// ---------------------------------------------------------------------------------------
template <int VEC, bool FOLD>
__global__ void __launch_bounds__(TX *TY) recombine2_kernel(const Node *__restrict__ parents, Bases bases, Regions2 reg,
                                                            int q, int item0, int peel, const Node *__restrict__ dfs_parents,
                                                            int fold, int fold_peel)
{
    using V = Vec<VEC>;
    using T = typename V::type;
    // last parent first: its products are the ones the preceding kernel wrote last, so they are still in L2
    const int par = item0 + (gridDim.z - 1 - blockIdx.z);
    const int c = (blockIdx.x * TX + threadIdx.x) * VEC;
    if (c >= q) return;
    const Operand cc = parents[par].c;
    double *C = resolve(bases, cc);
    const int64_t ldc = cc.ld, gld = reg.grand_ld;
    const double *grand = bases.p[BASE_WS] + reg.grand_q + int64_t(par) * 49 * reg.grand_mat;
    const int r0 = blockIdx.y * TILE_ROWS + threadIdx.y;
    FoldTarget ft{};
    if (FOLD) ft = fold_target(dfs_parents[par], bases, 4 * q, fold - 1, fold_peel);     // see recombine_bfs_kernel
    // peel != 0: parent of odd size 4q + 1; add A[row][4q] * B[4q][col] to every entry (see recombine_bfs_kernel)
    const double *acol = nullptr;
    int64_t lda = 0;
    T bv[4] = {T(), T(), T(), T()};
    if (peel) {
        const Operand pa = parents[par].a, pb = parents[par].b;
        acol = resolve(bases, pa) + 4 * q;
        lda = pa.ld;
        const double *brow = resolve(bases, pb) + int64_t(4 * q) * pb.ld + c;
#pragma unroll
        for (int t = 0; t < 4; ++t) bv[t] = V::ldk(brow + t * q);
    }
#pragma unroll 1
    for (int i = 0; i < ROWS_PER_THREAD; ++i) {
        const int r = r0 + i * TY;
        if (r >= q) break;
        const int64_t og = int64_t(r) * gld + c;
        T z[7][2][2];   // product of child j at quadrant position (u, v)
#pragma unroll
        for (int j = 0; j < 7; ++j) {
            const double *g = grand + int64_t(j) * 7 * reg.grand_mat + og;
            T k[7];
#pragma unroll
            for (int t = 0; t < 7; ++t) k[t] = V::ld(g + t * reg.grand_mat);
            const T u1 = V::add(k[0], k[3]);
            const T u2 = V::add(u1, k[4]);
            const T u3 = V::add(u1, k[2]);
            z[j][0][0] = V::add(k[0], k[1]);
            z[j][0][1] = V::add(u3, k[5]);
            z[j][1][0] = V::sub(u2, k[6]);
            z[j][1][1] = V::add(u2, k[2]);
        }
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int v = 0; v < 2; ++v) {
                const T u1 = V::add(z[0][u][v], z[3][u][v]);
                const T u2 = V::add(u1, z[4][u][v]);
                const T u3 = V::add(u1, z[2][u][v]);
                double *o = C + (int64_t(u) * q + r) * ldc + v * q + c;     // block (u, v) of C11
                const int64_t h = 2 * int64_t(q);
                T c11 = V::add(z[0][u][v], z[1][u][v]), c12 = V::add(u3, z[5][u][v]);
                T c21 = V::sub(u2, z[6][u][v]), c22 = V::add(u2, z[2][u][v]);
                if (peel) {
                    const double a0 = acol[(int64_t(u) * q + r) * lda], a1 = acol[(int64_t(u) * q + r + h) * lda];
                    c11 = V::fma1(a0, bv[v], c11); c12 = V::fma1(a0, bv[2 + v], c12);
                    c21 = V::fma1(a1, bv[v], c21); c22 = V::fma1(a1, bv[2 + v], c22);
                }
                if (FOLD) {
                    const int R = u * q + r, Cc = v * q + c;
                    fold_emit<VEC>(ft, R, Cc, c11);
                    fold_emit<VEC>(ft, R, Cc + int(h), c12);
                    fold_emit<VEC>(ft, R + int(h), Cc, c21);
                    fold_emit<VEC>(ft, R + int(h), Cc + int(h), c22);
                } else {
                    V::st(o, c11);
                    V::st(o + h, c12);
                    V::st(o + h * ldc, c21);
                    V::st(o + h * ldc + h, c22);
                }
            }
    }
}

// ---------------------------------------------------------------------------------------
// The two-level passes for children of ODD size h = 2q + 1 (parent m = 2h, children peeled, grandchildren q).
// Thread (r, c) with r, c <= q: for r, c < q it owns the 4 x 4 lattice of parent positions whose child-local
// rows are {r, q + r} and columns {c, q + c} -- exactly the even pass, except that a child's quadrants start at
// h, not 2q; a thread with r = q (c = q) owns the children's peeled row (column) 2q instead.  Differences from
// the even pass: the children's sums are written in all four quadrants and on the peeled row and column (their
// own peeling fix-ups read the whole operands); in the recombination every child's product gets the rank-one
// term of its peeled split, Acol_j[row] * Brow_j[col], before the parent's U-chain, and the children's last row
// and column -- thin products written into their Q slots beforehand -- are read from memory by the edge threads.
// Same operations in the same order per element as one pass per level.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void child_sums(int side, double x11, double x12, double x21, double x22, double (&y)[7], double (&s)[4])
{
    if (side == 0) {
        s[0] = x21 + x22;       // T2
        s[1] = s[0] - x11;      // T3
        s[2] = x11 - x21;       // T4
        s[3] = x12 - s[1];      // T5
        y[0] = x11; y[1] = x12; y[2] = s[0]; y[3] = s[1]; y[4] = s[2]; y[5] = s[3]; y[6] = x22;
    } else {
        s[0] = x12 - x11;       // S2
        s[1] = x22 - s[0];      // S3
        s[2] = x22 - x12;       // S4
        s[3] = s[1] - x21;      // S6
        y[0] = x11; y[1] = x21; y[2] = s[0]; y[3] = s[1]; y[4] = s[2]; y[5] = x22; y[6] = s[3];
    }
}

__global__ void __launch_bounds__(TX *TY) form2_odd_kernel(const Node *__restrict__ parents, Bases bases, Regions2 reg, int q, int item0)
{
    const int item = item0 + blockIdx.z;
    const int par = item >> 1, side = item & 1;
    const int c = blockIdx.x * TX + threadIdx.x, r = blockIdx.y * TY + threadIdx.y;
    if (c > q || r > q) return;
    const int h = 2 * q + 1;
    const Operand x = side ? parents[par].b : parents[par].a;
    const double *X = resolve(bases, x);
    const int64_t ld = x.ld;
    double *ws = bases.p[BASE_WS];
    double *child = ws + (side ? reg.child_s : reg.child_t) + int64_t(par) * 4 * reg.child_mat;
    double *grand = ws + (side ? reg.grand_s : reg.grand_t) + int64_t(par) * 28 * reg.grand_mat;
    const int64_t cld = reg.child_ld, gld = reg.grand_ld;
    const int nr = r < q ? 2 : 1, nc = c < q ? 2 : 1;
    double y[7][2][2];
    // all loads of the thread first (up to 16), then the sums
    double xv[2][2][4];
#pragma unroll
    for (int u = 0; u < 2; ++u)
#pragma unroll
        for (int v = 0; v < 2; ++v) {
            if (u >= nr || v >= nc) continue;
            const int cr = r < q ? u * q + r : 2 * q, cc = c < q ? v * q + c : 2 * q;      // position inside the child
            const double *p = X + int64_t(cr) * ld + cc;
            xv[u][v][0] = __ldcs(p);
            xv[u][v][1] = __ldcs(p + h);
            xv[u][v][2] = __ldcs(p + int64_t(h) * ld);
            xv[u][v][3] = __ldcs(p + int64_t(h) * ld + h);
        }
#pragma unroll
    for (int u = 0; u < 2; ++u)
#pragma unroll
        for (int v = 0; v < 2; ++v) {
            if (u >= nr || v >= nc) continue;
            const int cr = r < q ? u * q + r : 2 * q, cc = c < q ? v * q + c : 2 * q;
            double yy[7], ss[4];
            child_sums(side, xv[u][v][0], xv[u][v][1], xv[u][v][2], xv[u][v][3], yy, ss);
#pragma unroll
            for (int j = 0; j < 7; ++j) y[j][u][v] = yy[j];
            const int64_t o = int64_t(cr) * cld + cc;
#pragma unroll
            for (int k = 0; k < 4; ++k) child[k * reg.child_mat + o] = ss[k];
        }
    if (r >= q || c >= q) return;
    const int64_t og = int64_t(r) * gld + c;
#pragma unroll
    for (int j = 0; j < 7; ++j) {
        double yy[7], ss[4];
        child_sums(side, y[j][0][0], y[j][0][1], y[j][1][0], y[j][1][1], yy, ss);
        double *g = grand + int64_t(j) * 4 * reg.grand_mat + og;
#pragma unroll
        for (int k = 0; k < 4; ++k) g[k * reg.grand_mat] = ss[k];
    }
}

__device__ __forceinline__ void u_chain7(const double (&k)[7], double &c11, double &c12, double &c21, double &c22)
{
    const double u1 = k[0] + k[3], u2 = u1 + k[4], u3 = u1 + k[2];
    c11 = k[0] + k[1];
    c12 = u3 + k[5];
    c21 = u2 - k[6];
    c22 = u2 + k[2];
}

__global__ void __launch_bounds__(TX *TY) recombine2_odd_kernel(const Node *__restrict__ parents, const Node *__restrict__ children,
                                                                Bases bases, Regions2 reg, int q, int item0, int peel)
{
    // last parent first: its products are the ones the preceding kernel wrote last, so they are still in L2
    const int par = item0 + (gridDim.z - 1 - blockIdx.z);
    const int c = blockIdx.x * TX + threadIdx.x, r = blockIdx.y * TY + threadIdx.y;
    if (c > q || r > q) return;
    const int h = 2 * q + 1;
    const Node *kids = children + size_t(par) * 7;
    const Operand cc_op = parents[par].c;
    double *C = resolve(bases, cc_op);
    const int64_t ldc = cc_op.ld, gld = reg.grand_ld;
    // peel != 0: the parent itself is odd (size 2h + 1): every entry also gets A[row][2h] * B[2h][col]
    const double *pacol = nullptr, *pbrow = nullptr;
    int64_t plda = 0;
    if (peel) {
        const Operand pa = parents[par].a, pb = parents[par].b;
        pacol = resolve(bases, pa) + 2 * h;
        plda = pa.ld;
        pbrow = resolve(bases, pb) + int64_t(2 * h) * pb.ld;
    }
    auto emit = [&](int cr, int ccol, const double (&z)[7]) {       // the seven child products at child position (cr, ccol)
        double v[4];
        u_chain7(z, v[0], v[1], v[2], v[3]);
#pragma unroll
        for (int quad = 0; quad < 4; ++quad) {
            const int R = cr + (quad >> 1) * h, Cc = ccol + (quad & 1) * h;
            double val = v[quad];
            if (peel) val = fma(pacol[int64_t(R) * plda], pbrow[Cc], val);
            C[int64_t(R) * ldc + Cc] = val;
        }
    };
    if (r < q && c < q) {
        const double *grand = bases.p[BASE_WS] + reg.grand_q + int64_t(par) * 49 * reg.grand_mat + int64_t(r) * gld + c;
        double z[7][2][2];
#pragma unroll
        for (int j = 0; j < 7; ++j) {
            const double *g = grand + int64_t(j) * 7 * reg.grand_mat;
            double k[7];
#pragma unroll
            for (int t = 0; t < 7; ++t) k[t] = __ldcs(g + t * reg.grand_mat);
            u_chain7(k, z[j][0][0], z[j][0][1], z[j][1][0], z[j][1][1]);
            // the rank-one term of child j's own peeled split: its operands' column 2q and row 2q
            const Operand ka = kids[j].a, kb = kids[j].b;
            const double *acol = resolve(bases, ka) + 2 * q, *brow = resolve(bases, kb) + int64_t(2 * q) * kb.ld;
            const double a0 = acol[int64_t(r) * ka.ld], a1 = acol[int64_t(q + r) * ka.ld], b0 = brow[c], b1 = brow[q + c];
            z[j][0][0] = fma(a0, b0, z[j][0][0]);
            z[j][0][1] = fma(a0, b1, z[j][0][1]);
            z[j][1][0] = fma(a1, b0, z[j][1][0]);
            z[j][1][1] = fma(a1, b1, z[j][1][1]);
        }
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int v = 0; v < 2; ++v) {
                const double zz[7] = {z[0][u][v], z[1][u][v], z[2][u][v], z[3][u][v], z[4][u][v], z[5][u][v], z[6][u][v]};
                emit(u * q + r, v * q + c, zz);
            }
        return;
    }
    // the children's peeled row (r = q) and column (c = q): their products were written by the thin products
    const int nr = r < q ? 2 : 1, nc = c < q ? 2 : 1;
    for (int u = 0; u < nr; ++u)
        for (int v = 0; v < nc; ++v) {
            const int cr = r < q ? u * q + r : 2 * q, ccol = c < q ? v * q + c : 2 * q;
            double zz[7];
#pragma unroll
            for (int j = 0; j < 7; ++j) {
                const Operand kc = kids[j].c;
                zz[j] = resolve(bases, kc)[int64_t(cr) * kc.ld + ccol];
            }
            emit(cr, ccol, zz);
        }
}

// ---------------------------------------------------------------------------------------
// Peeling fix-ups for an odd node size m = e + 1 (block algebra on the split
// A = [A1 ac; ar al], B = [B1 bc; br be]):  the recursion has produced A1.B1 in C[0:e,0:e].
//   rank-one:    C[r][c] += A[r][e] * B[e][c]            r, c < e
//   last column: C[r][e]  = sum_k A[r][k] * B[k][e]      r < m
//   last row:    C[e][c]  = sum_k A[e][k] * B[k][c]      c < e
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) peel_rank1_kernel(const Node *__restrict__ nodes, Bases bases, int e, int item0)
{
    const Node nd = nodes[item0 + blockIdx.z];
    const int c = blockIdx.x * 64 + threadIdx.x;
    if (c >= e) return;
    const double *A = resolve(bases, nd.a), *B = resolve(bases, nd.b);
    double *C = resolve(bases, nd.c);
    const double b = B[int64_t(e) * nd.b.ld + c];
    const int r0 = blockIdx.y * TILE_ROWS + threadIdx.y;
#pragma unroll
    for (int i = 0; i < ROWS_PER_THREAD; ++i) {
        const int r = r0 + i * TY;
        if (r < e) {
            double *o = C + int64_t(r) * nd.c.ld + c;
            *o = fma(A[int64_t(r) * nd.a.ld + e], b, *o);
        }
    }
}

// Thin products: a few columns or a few rows of C = A.B of one node, over the full inner
// dimension K.  They serve the peeled last column / row (one of each) and the ragged remainder of
// base products whose size is a few elements past a multiple of the GEMM tile (e.g. 771 = 768 + 3).
// Both read one operand in full exactly once and are bound by that stream from HBM.  They run on the FP64
// tensor cores with the operand fragments loaded straight from global memory in the layout mma.sync
// m8n8k4 wants (no shared-memory staging): a lane's 8-byte load of the large operand shares its 32-byte
// sector with the three lanes next to it, so every sector fetched is used in full, and 8 to 16 such loads
// per lane are in flight before the first DMMA.  Summation runs over k ascending: bit-reproducible.
__device__ __forceinline__ void dmma_thin(double &d0, double &d1, double a, double b)
{
    asm("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};\n"
        : "+d"(d0), "+d"(d1)
        : "d"(a), "d"(b));
}

constexpr int THIN_WARPS = 4;      // warps per CTA.  THIN_STEPS = 4-deep steps per loop iteration: 8, or 16 for launches
                                   // over a few nodes only, whose few warps need more loads in flight each

// Columns [c0, c0 + nc) of C for rows [0, rows), nc <= 8: a warp owns 8 rows.  g = lane / 4, q = lane % 4:
// the lane feeds A[row g][k + q] and B[k + q][column g] and receives C[row g][columns 2q, 2q + 1].
// KSPLIT (launches over one or two nodes, which would leave each SM a handful of warps): the CTA owns 8 rows, its
// warps take the chunks of the inner dimension in turn and warp 0 adds their sums in warp order.
template <int THIN_STEPS, bool KSPLIT = false>
__global__ void __launch_bounds__(THIN_WARPS * 32) thin_cols_kernel(const Node *__restrict__ nodes, Bases bases, int K, int rows,
                                                                    int c0, int nc, int item0)
{
    __shared__ double part[KSPLIT ? THIN_WARPS - 1 : 1][2][32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, q = lane & 3;
    const int m0 = KSPLIT ? blockIdx.x * 8 : (blockIdx.x * THIN_WARPS + warp) * 8;
    if (!KSPLIT && m0 >= rows) return;
    const Node nd = nodes[item0 + blockIdx.y];
    const double *A = resolve(bases, nd.a), *B = resolve(bases, nd.b);
    const bool row_ok = m0 + g < rows, col_ok = g < nc;
    const double *a = A + int64_t(row_ok ? m0 + g : 0) * nd.a.ld + q;
    const double *b = B + int64_t(q) * nd.b.ld + c0 + (col_ok ? g : 0);
    const int64_t ldb = nd.b.ld;
    double d0 = 0.0, d1 = 0.0;
    for (int k0 = KSPLIT ? warp * 4 * THIN_STEPS : 0; k0 < K; k0 += (KSPLIT ? THIN_WARPS : 1) * 4 * THIN_STEPS) {
        double av[THIN_STEPS], bv[THIN_STEPS];
        if (k0 + 4 * THIN_STEPS <= K) {
#pragma unroll
            for (int s = 0; s < THIN_STEPS; ++s) av[s] = row_ok ? __ldcs(a + k0 + 4 * s) : 0.0;
#pragma unroll
            for (int s = 0; s < THIN_STEPS; ++s) bv[s] = col_ok ? b[int64_t(k0 + 4 * s) * ldb] : 0.0;
        } else {
#pragma unroll
            for (int s = 0; s < THIN_STEPS; ++s) {
                const bool k_ok = k0 + 4 * s + q < K;
                av[s] = row_ok && k_ok ? __ldcs(a + k0 + 4 * s) : 0.0;
                bv[s] = col_ok && k_ok ? b[int64_t(k0 + 4 * s) * ldb] : 0.0;
            }
        }
#pragma unroll
        for (int s = 0; s < THIN_STEPS; ++s) dmma_thin(d0, d1, av[s], bv[s]);
    }
    if (KSPLIT) {
        if (warp > 0) {
            part[warp - 1][0][lane] = d0;
            part[warp - 1][1][lane] = d1;
        }
        __syncthreads();
        if (warp > 0) return;
#pragma unroll
        for (int w = 0; w < THIN_WARPS - 1; ++w) {
            d0 += part[w][0][lane];
            d1 += part[w][1][lane];
        }
    }
    if (row_ok) {
        double *o = resolve(bases, nd.c) + int64_t(m0 + g) * nd.c.ld + c0 + 2 * q;
        if (2 * q < nc) o[0] = d0;
        if (2 * q + 1 < nc) o[1] = d1;
    }
}

// Rows [r0, r0 + nr) of C for columns [0, cols), nr <= 8: a warp owns NT adjacent groups of 8 columns.  The lane
// feeds A[r0 + g][k + q] (zero for g >= nr) and B[k + q][column g of each group].
template <int NT, int THIN_STEPS, bool KSPLIT = false>
__global__ void __launch_bounds__(THIN_WARPS * 32) thin_rows_kernel(const Node *__restrict__ nodes, Bases bases, int K, int cols,
                                                                    int r0, int nr, int item0)
{
    __shared__ double part[KSPLIT ? THIN_WARPS - 1 : 1][2 * NT][32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, q = lane & 3;
    const int n0 = KSPLIT ? blockIdx.x * 8 * NT : (blockIdx.x * THIN_WARPS + warp) * 8 * NT;
    if (!KSPLIT && n0 >= cols) return;
    const Node nd = nodes[item0 + blockIdx.y];
    const double *A = resolve(bases, nd.a), *B = resolve(bases, nd.b);
    const bool row_ok = g < nr;
    const double *a = A + int64_t(r0 + (row_ok ? g : 0)) * nd.a.ld + q;
    const int64_t ldb = nd.b.ld;
    bool col_ok[NT];
    const double *b[NT];
#pragma unroll
    for (int j = 0; j < NT; ++j) {
        col_ok[j] = n0 + 8 * j + g < cols;
        b[j] = B + int64_t(q) * ldb + (col_ok[j] ? n0 + 8 * j + g : 0);
    }
    double d[NT][2];
#pragma unroll
    for (int j = 0; j < NT; ++j) d[j][0] = d[j][1] = 0.0;
    for (int k0 = KSPLIT ? warp * 4 * THIN_STEPS : 0; k0 < K; k0 += (KSPLIT ? THIN_WARPS : 1) * 4 * THIN_STEPS) {
        double av[THIN_STEPS], bv[THIN_STEPS][NT];
        const bool full = k0 + 4 * THIN_STEPS <= K;
#pragma unroll
        for (int s = 0; s < THIN_STEPS; ++s) {
            const bool k_ok = full || k0 + 4 * s + q < K;
#pragma unroll
            for (int j = 0; j < NT; ++j) bv[s][j] = col_ok[j] && k_ok ? __ldcs(b[j] + int64_t(k0 + 4 * s) * ldb) : 0.0;
            av[s] = row_ok && k_ok ? a[k0 + 4 * s] : 0.0;
        }
#pragma unroll
        for (int s = 0; s < THIN_STEPS; ++s)
#pragma unroll
            for (int j = 0; j < NT; ++j) dmma_thin(d[j][0], d[j][1], av[s], bv[s][j]);
    }
    if (KSPLIT) {
        if (warp > 0) {
#pragma unroll
            for (int j = 0; j < NT; ++j) {
                part[warp - 1][2 * j][lane] = d[j][0];
                part[warp - 1][2 * j + 1][lane] = d[j][1];
            }
        }
        __syncthreads();
        if (warp > 0) return;
#pragma unroll
        for (int w = 0; w < THIN_WARPS - 1; ++w)
#pragma unroll
            for (int j = 0; j < NT; ++j) {
                d[j][0] += part[w][2 * j][lane];
                d[j][1] += part[w][2 * j + 1][lane];
            }
    }
    if (row_ok) {
        double *o = resolve(bases, nd.c) + int64_t(r0 + g) * nd.c.ld;
#pragma unroll
        for (int j = 0; j < NT; ++j) {
            const int c = n0 + 8 * j + 2 * q;
            if (c < cols) o[c] = d[j][0];
            if (c + 1 < cols) o[c + 1] = d[j][1];
        }
    }
}

// The same thin products for the seven children of one BFS parent at once.  Their large operands are the sums
// T_0 .. T_6 (S_0 .. S_6) of the parent's four quadrants (Appendix A), so a pass that reads the four quadrants and
// forms the seven fragments in registers moves 4 h^2 words per parent where seven separate thin products read
// 7 h^2.  The small operand (the children's own last columns of S_j, last rows of T_j) and the outputs belong to
// the children: child j of parent p is leaves[7 p + j].  The sums are formed in the order of the formation
// kernels, so every product sees the values those kernels stored.
constexpr int SIB_STEPS = 4;       // 4-deep steps per loop iteration: 16 quadrant loads and 28 small loads in flight per lane.
// The two kernels run at 3.6 and 4.4 TB/s, bound by the latency of those loads at 12 to 16 warps per SM.  Measured and not
// kept (n = 12345; leaves' remainders + peeled level 3 = 5.8 ms per product as is): 8 steps in registers (peel 3.0 -> 5.1 ms);
// the seven small vectors of a peeled level staged in shared memory (6.1 ms); the quadrant streams through a per-warp
// ring of 8-byte cp.async copies, three chunks in flight (peel 4.2 ms, remainders +0.8 ms: 8-byte asynchronous copies are
// slower than plain loads); the inner dimension split over the warps of a CTA (peel 2.9 ms, remainders +0.2 ms, and a
// summation order of its own); the small operand loaded once per CTA and chunk by all threads together and handed over through
// shared memory, one barrier per chunk (peel 3.1 ms, remainders +0.4 ms); 96 or 128 registers for more warps per SM, and plain
// instead of streaming loads (no gain).  Counters at 49 parents of 771: DRAM 47 %, L2 44 %, L1 data pipe 56 %, DMMA 38 %,
// 10.7 warps active per SM, long-scoreboard stalls: no unit is saturated, the loop waits on its loads.

// Columns [c0, c0 + nc) of the children's products, all h rows: a warp owns 8 rows of all seven.  Summation over k ascending,
// like the per-leaf kernels: plans that differ only in which of the two serves a node give the same bits.
__global__ void __launch_bounds__(THIN_WARPS * 32) thin_cols_siblings_kernel(const Node *__restrict__ parents, const Node *__restrict__ leaves,
                                                                             Bases bases, int h, int c0, int nc, int item0)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, q = lane & 3;
    const int m0 = (blockIdx.x * THIN_WARPS + warp) * 8;
    if (m0 >= h) return;
    const int64_t p = item0 + blockIdx.y;
    const Node par = parents[p];
    const Node *kid = leaves + 7 * p;
    const bool row_ok = m0 + g < h, col_ok = g < nc;
    const int64_t lda = par.a.ld;
    const double *x11 = resolve(bases, par.a) + int64_t(row_ok ? m0 + g : 0) * lda + q;
    const double *x21 = x11 + int64_t(h) * lda;
    const double *b[7];
    int64_t ldb[7];
#pragma unroll
    for (int j = 0; j < 7; ++j) {
        const Operand o = kid[j].b;
        ldb[j] = o.ld;
        b[j] = resolve(bases, o) + int64_t(q) * o.ld + c0 + (col_ok ? g : 0);
    }
    double d[7][2];
#pragma unroll
    for (int j = 0; j < 7; ++j) d[j][0] = d[j][1] = 0.0;
    for (int k0 = 0; k0 < h; k0 += 4 * SIB_STEPS) {
        double x[SIB_STEPS][4], bv[SIB_STEPS][7];
        const bool full = k0 + 4 * SIB_STEPS <= h;
#pragma unroll
        for (int s = 0; s < SIB_STEPS; ++s) {
            const int k = k0 + 4 * s;
            const bool k_ok = full || k + q < h;
            const bool ok = row_ok && k_ok;
            x[s][0] = ok ? __ldcs(x11 + k) : 0.0;
            x[s][1] = ok ? __ldcs(x11 + h + k) : 0.0;
            x[s][2] = ok ? __ldcs(x21 + k) : 0.0;
            x[s][3] = ok ? __ldcs(x21 + h + k) : 0.0;
#pragma unroll
            for (int j = 0; j < 7; ++j) bv[s][j] = col_ok && k_ok ? b[j][int64_t(k) * ldb[j]] : 0.0;
        }
#pragma unroll
        for (int s = 0; s < SIB_STEPS; ++s) {
            const double t2 = x[s][2] + x[s][3], t3 = t2 - x[s][0], t4 = x[s][0] - x[s][2], t5 = x[s][1] - t3;
            dmma_thin(d[0][0], d[0][1], x[s][0], bv[s][0]);
            dmma_thin(d[1][0], d[1][1], x[s][1], bv[s][1]);
            dmma_thin(d[2][0], d[2][1], t2, bv[s][2]);
            dmma_thin(d[3][0], d[3][1], t3, bv[s][3]);
            dmma_thin(d[4][0], d[4][1], t4, bv[s][4]);
            dmma_thin(d[5][0], d[5][1], t5, bv[s][5]);
            dmma_thin(d[6][0], d[6][1], x[s][3], bv[s][6]);
        }
    }
    if (row_ok) {
#pragma unroll
        for (int j = 0; j < 7; ++j) {
            const Operand c = kid[j].c;
            double *o = resolve(bases, c) + int64_t(m0 + g) * c.ld + c0 + 2 * q;
            if (2 * q < nc) o[0] = d[j][0];
            if (2 * q + 1 < nc) o[1] = d[j][1];
        }
    }
}

// Rows [r0, r0 + nr) of the children's products, columns [0, cols): a warp owns 8 columns of all seven.
__global__ void __launch_bounds__(THIN_WARPS * 32) thin_rows_siblings_kernel(const Node *__restrict__ parents, const Node *__restrict__ leaves,
                                                                             Bases bases, int h, int cols, int r0, int nr, int item0)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, q = lane & 3;
    const int n0 = (blockIdx.x * THIN_WARPS + warp) * 8;
    if (n0 >= cols) return;
    const int64_t p = item0 + blockIdx.y;
    const Node par = parents[p];
    const Node *kid = leaves + 7 * p;
    const bool row_ok = g < nr, col_ok = n0 + g < cols;
    const int64_t ldb = par.b.ld;
    const double *y11 = resolve(bases, par.b) + int64_t(q) * ldb + (col_ok ? n0 + g : 0);
    const double *y21 = y11 + int64_t(h) * ldb;
    const double *a[7];
#pragma unroll
    for (int j = 0; j < 7; ++j) {
        const Operand o = kid[j].a;
        a[j] = resolve(bases, o) + int64_t(r0 + (row_ok ? g : 0)) * o.ld + q;
    }
    double d[7][2];
#pragma unroll
    for (int j = 0; j < 7; ++j) d[j][0] = d[j][1] = 0.0;
    for (int k0 = 0; k0 < h; k0 += 4 * SIB_STEPS) {
        double y[SIB_STEPS][4], av[SIB_STEPS][7];
        const bool full = k0 + 4 * SIB_STEPS <= h;
#pragma unroll
        for (int s = 0; s < SIB_STEPS; ++s) {
            const int k = k0 + 4 * s;
            const bool k_ok = full || k + q < h;
            const bool ok = col_ok && k_ok;
            y[s][0] = ok ? __ldcs(y11 + int64_t(k) * ldb) : 0.0;
            y[s][1] = ok ? __ldcs(y11 + int64_t(k) * ldb + h) : 0.0;
            y[s][2] = ok ? __ldcs(y21 + int64_t(k) * ldb) : 0.0;
            y[s][3] = ok ? __ldcs(y21 + int64_t(k) * ldb + h) : 0.0;
#pragma unroll
            for (int j = 0; j < 7; ++j) av[s][j] = row_ok && k_ok ? a[j][k] : 0.0;
        }
#pragma unroll
        for (int s = 0; s < SIB_STEPS; ++s) {
            const double s2 = y[s][1] - y[s][0], s3 = y[s][3] - s2, s4 = y[s][3] - y[s][1], s6 = s3 - y[s][2];
            dmma_thin(d[0][0], d[0][1], av[s][0], y[s][0]);
            dmma_thin(d[1][0], d[1][1], av[s][1], y[s][2]);
            dmma_thin(d[2][0], d[2][1], av[s][2], s2);
            dmma_thin(d[3][0], d[3][1], av[s][3], s3);
            dmma_thin(d[4][0], d[4][1], av[s][4], s4);
            dmma_thin(d[5][0], d[5][1], av[s][5], y[s][3]);
            dmma_thin(d[6][0], d[6][1], av[s][6], s6);
        }
    }
    if (row_ok) {
#pragma unroll
        for (int j = 0; j < 7; ++j) {
            const Operand c = kid[j].c;
            double *o = resolve(bases, c) + int64_t(r0 + g) * c.ld;
            const int col = n0 + 2 * q;
            if (col < cols) o[col] = d[j][0];
            if (col + 1 < cols) o[col + 1] = d[j][1];
        }
    }
}

dim3 tile_grid(int64_t h, int vec, int64_t items)
{
    return dim3(unsigned((h + TX * vec - 1) / (TX * vec)), unsigned((h + TILE_ROWS - 1) / TILE_ROWS), unsigned(items));
}

// fewer than two CTAs per SM of a B200
bool small_grid(const dim3 &g) { return int64_t(g.x) * g.y * g.z < 2 * kNominalSMs; }

int chunks(int64_t items) { return int((items + MAX_Z - 1) / MAX_Z); }

}  // namespace

int launches_of(const Launch &op)
{
    switch (op.kind) {
    case OP_FORM: return chunks(op.count * 2);
    case OP_RECOMBINE: return chunks(op.count);
    case OP_FORM_ONE: return chunks(op.count * ((op.j >= 2 && op.j <= 4) ? 2 : 1));
    case OP_ACCUMULATE: return chunks(op.count);
    case OP_PEEL:
        return (op.peel_fused ? 0 : chunks(op.count)) + 2 * chunks(op.sibling_tab > 0 && op.count % 7 == 0 ? op.count / 7 : op.count);
    case OP_GEMM: {
        const int rem = gemm_thin_remainder(op.m), bulk = int(op.m) - rem;
        int tiled = 0;
        if (bulk > 0) {
            GemmRegion regions[4];
            tiled = gemm_regions(bulk, op.count, kNominalSMs, regions);
        }
        return tiled + (rem ? chunks(gemm_thin_siblings(op) ? op.count / 7 : op.count) * (bulk > 0 ? 2 : 1) : 0);
    }
    case OP_FORM2: return chunks(op.count * 2);
    case OP_RECOMBINE2: return chunks(op.count);
    case OP_FORM2_ODD: return chunks(op.count * 2);
    case OP_RECOMBINE2_ODD: return chunks(op.count);
    case OP_FORM3: return chunks(op.count * 2);
    case OP_RECOMBINE3: return chunks(op.count);
    case OP_FUSED_STEP: return chunks(op.count);
    case OP_LINCOMB: return chunks(op.count);
    }
    return 0;
}

#define FOR_CHUNKS(total)                                              \
    for (int64_t item0 = 0, zn; item0 < (total); item0 += MAX_Z)       \
        if ((zn = ((total) - item0 < MAX_Z ? (total) - item0 : MAX_Z)), true)

cudaError_t launch_form(const Node *tab, const Launch &op, const Bases &bases, bool vec, cudaStream_t stream,
                        int *launched)
{
    const dim3 block(TX, TY);
    const int64_t total = op.count * 2;
    FOR_CHUNKS(total) {
        const int v = vec ? 2 : 1;
        const dim3 grid = tile_grid(op.h, v, zn);
        const Node *par = tab + op.parent_tab, *kid = tab + op.child_tab;
        if (small_grid(grid)) {          // too few CTAs to fill the SMs: one row per thread, four times the CTAs
            const dim3 g1(grid.x, unsigned((op.h + TY - 1) / TY), grid.z);
            if (vec) form_bfs_kernel<2, 1><<<g1, block, 0, stream>>>(par, kid, bases, int(op.h), int(item0));
            else form_bfs_kernel<1, 1><<<g1, block, 0, stream>>>(par, kid, bases, int(op.h), int(item0));
        } else {
            if (vec) form_bfs_kernel<2, ROWS_PER_THREAD><<<grid, block, 0, stream>>>(par, kid, bases, int(op.h), int(item0));
            else form_bfs_kernel<1, ROWS_PER_THREAD><<<grid, block, 0, stream>>>(par, kid, bases, int(op.h), int(item0));
        }
        ++*launched;
    }
    return cudaGetLastError();
}

template <int VEC, int RPT>
void launch_recombine_as(const dim3 &grid, const dim3 &block, cudaStream_t stream, const Node *tab, const Launch &op, const Bases &bases,
                         int64_t item0)
{
    const Node *par = tab + op.parent_tab, *kid = tab + op.child_tab;
    if (op.fold && op.fold_tolerant && VEC == 2)
        recombine_bfs_kernel<VEC, RPT, 2><<<grid, block, 0, stream>>>(par, kid, bases, int(op.h), int(item0), op.peel_fused,
                                                                     tab + op.fold_tab, op.fold, op.fold_peel);
    else if (op.fold)
        recombine_bfs_kernel<VEC, RPT, 1><<<grid, block, 0, stream>>>(par, kid, bases, int(op.h), int(item0), op.peel_fused,
                                                                     tab + op.fold_tab, op.fold, op.fold_peel);
    else
        recombine_bfs_kernel<VEC, RPT, 0><<<grid, block, 0, stream>>>(par, kid, bases, int(op.h), int(item0), op.peel_fused, nullptr, 0, 0);
}

cudaError_t launch_recombine(const Node *tab, const Launch &op, const Bases &bases, bool vec, cudaStream_t stream,
                             int *launched)
{
    const dim3 block(TX, TY);
    const int64_t total = op.count;
    FOR_CHUNKS(total) {
        const int v = vec ? 2 : 1;
        const dim3 grid = tile_grid(op.h, v, zn);
        // folding passes also take one row per thread: their read-modify-write of C is a second round trip to memory
        // behind the loads of the products, and four times the CTAs keep enough of both in flight
        if (small_grid(grid) || op.fold) {
            const dim3 g1(grid.x, unsigned((op.h + TY - 1) / TY), grid.z);
            if (vec) launch_recombine_as<2, 1>(g1, block, stream, tab, op, bases, item0);
            else launch_recombine_as<1, 1>(g1, block, stream, tab, op, bases, item0);
        } else {
            if (vec) launch_recombine_as<2, ROWS_PER_THREAD>(grid, block, stream, tab, op, bases, item0);
            else launch_recombine_as<1, ROWS_PER_THREAD>(grid, block, stream, tab, op, bases, item0);
        }
        ++*launched;
    }
    return cudaGetLastError();
}

cudaError_t launch_form2(const Node *tab, const Launch &op, const Bases &bases, bool vec, cudaStream_t stream, int *launched)
{
    const dim3 block(TX, TY);
    const int64_t total = op.count * 2, q = op.h / 2;
    FOR_CHUNKS(total) {
        if (vec)
            form2_kernel<2><<<tile_grid(q, 2, zn), block, 0, stream>>>(tab + op.parent_tab, bases, op.reg, int(q), int(item0));
        else
            form2_kernel<1><<<tile_grid(q, 1, zn), block, 0, stream>>>(tab + op.parent_tab, bases, op.reg, int(q), int(item0));
        ++*launched;
    }
    return cudaGetLastError();
}

template <int VEC>
void launch_recombine2_as(const dim3 &grid, const dim3 &block, cudaStream_t stream, const Node *tab, const Launch &op, const Bases &bases,
                          int64_t q, int64_t item0)
{
    if (op.fold)
        recombine2_kernel<VEC, true><<<grid, block, 0, stream>>>(tab + op.parent_tab, bases, op.reg, int(q), int(item0), op.peel_fused,
                                                                tab + op.fold_tab, op.fold, op.fold_peel);
    else
        recombine2_kernel<VEC, false><<<grid, block, 0, stream>>>(tab + op.parent_tab, bases, op.reg, int(q), int(item0), op.peel_fused,
                                                                 nullptr, 0, 0);
}

cudaError_t launch_recombine2(const Node *tab, const Launch &op, const Bases &bases, bool vec, cudaStream_t stream,
                              int *launched)
{
    const dim3 block(TX, TY);
    const int64_t total = op.count, q = op.h / 2;
    FOR_CHUNKS(total) {
        if (vec) launch_recombine2_as<2>(tile_grid(q, 2, zn), block, stream, tab, op, bases, q, item0);
        else launch_recombine2_as<1>(tile_grid(q, 1, zn), block, stream, tab, op, bases, q, item0);
        ++*launched;
    }
    return cudaGetLastError();
}

cudaError_t launch_form2_odd(const Node *tab, const Launch &op, const Bases &bases, cudaStream_t stream, int *launched)
{
    const dim3 block(TX, TY);
    const int64_t total = op.count * 2, q = op.h / 2;       // op.h = 2q + 1
    FOR_CHUNKS(total) {
        const dim3 grid(unsigned((q + 1 + TX - 1) / TX), unsigned((q + 1 + TY - 1) / TY), unsigned(zn));
        form2_odd_kernel<<<grid, block, 0, stream>>>(tab + op.parent_tab, bases, op.reg, int(q), int(item0));
        ++*launched;
    }
    return cudaGetLastError();
}

cudaError_t launch_recombine2_odd(const Node *tab, const Launch &op, const Bases &bases, cudaStream_t stream, int *launched)
{
    const dim3 block(TX, TY);
    const int64_t total = op.count, q = op.h / 2;
    FOR_CHUNKS(total) {
        const dim3 grid(unsigned((q + 1 + TX - 1) / TX), unsigned((q + 1 + TY - 1) / TY), unsigned(zn));
        recombine2_odd_kernel<<<grid, block, 0, stream>>>(tab + op.parent_tab, tab + op.child_tab, bases, op.reg, int(q), int(item0),
                                                          op.peel_fused);
        ++*launched;
    }
    return cudaGetLastError();
}

cudaError_t launch_form_one(const Node *tab, const Launch &op, const Bases &bases, bool vec, cudaStream_t stream,
                            int *launched)
{
    const dim3 block(TX, TY);
    const int j = op.j;
    const int sides = (j >= 2 && j <= 5 ? 1 : 0) | ((j >= 2 && j <= 4) || j == 6 ? 2 : 0);
    if (sides == 0) return cudaSuccess;
    const int64_t total = op.count * (sides == 3 ? 2 : 1);
    FOR_CHUNKS(total) {
        if (vec)
            form_one_kernel<2><<<tile_grid(op.h, 2, zn), block, 0, stream>>>(tab + op.parent_tab, tab + op.child_tab,
                                                                            bases, int(op.h), j, sides, int(item0), op.chain);
        else
            form_one_kernel<1><<<tile_grid(op.h, 1, zn), block, 0, stream>>>(tab + op.parent_tab, tab + op.child_tab,
                                                                            bases, int(op.h), j, sides, int(item0), op.chain);
        ++*launched;
    }
    return cudaGetLastError();
}

cudaError_t launch_accumulate(const Node *tab, const Launch &op, const Bases &bases, bool vec, cudaStream_t stream,
                              int *launched)
{
    const dim3 block(TX, TY);
    const int64_t total = op.count;
    FOR_CHUNKS(total) {
        if (vec)
            accumulate_kernel<2><<<tile_grid(op.h, 2, zn), block, 0, stream>>>(
                tab + op.parent_tab, tab + op.child_tab, bases, int(op.h), op.j, int(item0), op.peel_fused);
        else
            accumulate_kernel<1><<<tile_grid(op.h, 1, zn), block, 0, stream>>>(
                tab + op.parent_tab, tab + op.child_tab, bases, int(op.h), op.j, int(item0), op.peel_fused);
        ++*launched;
    }
    return cudaGetLastError();
}

cudaError_t launch_thin_cols(const Node *nodes, const Bases &bases, int K, int rows, int c0, int nc, int64_t count,
                             cudaStream_t stream, int *launched)
{
    const int64_t total = count;
    FOR_CHUNKS(total) {
        const dim3 grid((rows + 8 * THIN_WARPS - 1) / (8 * THIN_WARPS), unsigned(zn));
        if (int64_t(grid.x) * zn < 4 * int64_t(kNominalSMs) && K >= 4096)
            thin_cols_kernel<8, true><<<dim3((rows + 7) / 8, unsigned(zn)), THIN_WARPS * 32, 0, stream>>>(nodes, bases, K, rows, c0, nc, int(item0));
        else if (int64_t(grid.x) * zn < 8 * int64_t(kNominalSMs)) thin_cols_kernel<16><<<grid, THIN_WARPS * 32, 0, stream>>>(nodes, bases, K, rows, c0, nc, int(item0));
        else thin_cols_kernel<8><<<grid, THIN_WARPS * 32, 0, stream>>>(nodes, bases, K, rows, c0, nc, int(item0));
        ++*launched;
    }
    return cudaGetLastError();
}

cudaError_t launch_thin_rows(const Node *nodes, const Bases &bases, int K, int cols, int r0, int nr, int64_t count,
                             cudaStream_t stream, int *launched)
{
    const int64_t total = count;
    // two groups of 8 columns per warp (128-byte runs of B) where that still leaves every SM a few dozen warps
    const bool two = (int64_t(cols + 15) / 16) * count >= 32 * int64_t(kNominalSMs);
    FOR_CHUNKS(total) {
        if (two) {
            const dim3 grid((cols + 16 * THIN_WARPS - 1) / (16 * THIN_WARPS), unsigned(zn));
            thin_rows_kernel<2, 8><<<grid, THIN_WARPS * 32, 0, stream>>>(nodes, bases, K, cols, r0, nr, int(item0));
        } else {
            const dim3 grid((cols + 8 * THIN_WARPS - 1) / (8 * THIN_WARPS), unsigned(zn));
            if (int64_t(grid.x) * zn < 4 * int64_t(kNominalSMs) && K >= 4096)
                thin_rows_kernel<1, 8, true><<<dim3((cols + 7) / 8, unsigned(zn)), THIN_WARPS * 32, 0, stream>>>(nodes, bases, K, cols, r0, nr, int(item0));
            else if (int64_t(grid.x) * zn < 8 * int64_t(kNominalSMs)) thin_rows_kernel<1, 16><<<grid, THIN_WARPS * 32, 0, stream>>>(nodes, bases, K, cols, r0, nr, int(item0));
            else thin_rows_kernel<1, 8><<<grid, THIN_WARPS * 32, 0, stream>>>(nodes, bases, K, cols, r0, nr, int(item0));
        }
        ++*launched;
    }
    return cudaGetLastError();
}

cudaError_t launch_thin_siblings(const Node *parents, const Node *leaves, const Bases &bases, int h, int M, int rem, int64_t count,
                                 cudaStream_t stream, int *launched)
{
    const int64_t total = count;       // parents; their children are leaves[7 p .. 7 p + 6]
    FOR_CHUNKS(total) {
        const dim3 grid((h + 8 * THIN_WARPS - 1) / (8 * THIN_WARPS), unsigned(zn));
        thin_cols_siblings_kernel<<<grid, THIN_WARPS * 32, 0, stream>>>(parents, leaves, bases, h, M, rem, int(item0));
        ++*launched;
    }
    if (M > 0) FOR_CHUNKS(total) {
        const dim3 grid((M + 8 * THIN_WARPS - 1) / (8 * THIN_WARPS), unsigned(zn));
        thin_rows_siblings_kernel<<<grid, THIN_WARPS * 32, 0, stream>>>(parents, leaves, bases, h, M, M, rem, int(item0));
        ++*launched;
    }
    return cudaGetLastError();
}

cudaError_t launch_peel(const Node *tab, const Launch &op, const Bases &bases, cudaStream_t stream, int *launched)
{
    const int m = int(op.m), e = m - 1;
    const Node *nodes = tab + op.parent_tab;
    const int64_t total = op.count;
    if (!op.peel_fused) {       // the recombination before this launch did not carry the rank-one term
        FOR_CHUNKS(total) {
            peel_rank1_kernel<<<dim3((e + 63) / 64, (e + TILE_ROWS - 1) / TILE_ROWS, unsigned(zn)), dim3(64, TY), 0,
                                stream>>>(nodes, bases, e, int(item0));
            ++*launched;
        }
    }
    if (op.sibling_tab > 0 && op.count % 7 == 0)      // seven siblings at a time, from their parent's quadrants
        return launch_thin_siblings(tab + (op.sibling_tab - 1), nodes, bases, m, e, 1, op.count / 7, stream, launched);
    cudaError_t err = launch_thin_cols(nodes, bases, m, m, e, 1, op.count, stream, launched);   // last column, all rows
    if (err != cudaSuccess) return err;
    return launch_thin_rows(nodes, bases, m, e, e, 1, op.count, stream, launched);              // last row, other columns
}

}  // namespace strassen
