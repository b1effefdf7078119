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

namespace strassen {

namespace {

constexpr int TX = 64, TY = 4, ROWS_PER_THREAD = 4, TILE_ROWS = TY * ROWS_PER_THREAD;
constexpr int MAX_Z = kMaxItemsPerLaunch;   // items per launch (gridDim.z limit is 65535)

template <int VEC> struct Vec;
template <> struct Vec<1> {
    using type = double;
    static __device__ __forceinline__ double ld(const double *p) { return __ldcs(p); }
    static __device__ __forceinline__ double ldk(const double *p) { return *p; }
    static __device__ __forceinline__ void st(double *p, double v) { *p = v; }
    static __device__ __forceinline__ double add(double a, double b) { return a + b; }
    static __device__ __forceinline__ double sub(double a, double b) { return a - b; }
    static __device__ __forceinline__ double neg(double a) { return -a; }
    static __device__ __forceinline__ double fma1(double a, double b, double v) { return fma(a, b, v); }
};
template <> struct Vec<2> {
    using type = double2;
    static __device__ __forceinline__ double2 ld(const double *p) { return __ldcs(reinterpret_cast<const double2 *>(p)); }
    static __device__ __forceinline__ double2 ldk(const double *p) { return *reinterpret_cast<const double2 *>(p); }
    static __device__ __forceinline__ void st(double *p, double2 v) { *reinterpret_cast<double2 *>(p) = v; }
    static __device__ __forceinline__ double2 add(double2 a, double2 b) { return make_double2(a.x + b.x, a.y + b.y); }
    static __device__ __forceinline__ double2 sub(double2 a, double2 b) { return make_double2(a.x - b.x, a.y - b.y); }
    static __device__ __forceinline__ double2 neg(double2 a) { return make_double2(-a.x, -a.y); }
    static __device__ __forceinline__ double2 fma1(double a, double2 b, double2 v) { return make_double2(fma(a, b.x, v.x), fma(a, b.y, v.y)); }
};

__device__ __forceinline__ double *resolve(const Bases &bases, const Operand &x) { return base_ptr(bases, x.base) + x.off; }

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
template <int VEC, int RPT>
__global__ void __launch_bounds__(TX *TY) recombine_bfs_kernel(const Node *__restrict__ parents,
                                                               const Node *__restrict__ children, Bases bases,
                                                               int h, int item0, int peel)
{
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
                V::st(o, c11);
                V::st(o + h, c12);
                V::st(o + hq, c21);
                V::st(o + hq + h, c22);
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
                                                          int j, int sides, int item0)
{
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
    const int which = side * 8 + j;
#pragma unroll
    for (int i = 0; i < ROWS_PER_THREAD; ++i) {
        const int r = r0 + i * TY;
        if (r >= h) continue;
        const double *q = X + int64_t(r) * ld + c;
        T v;
        switch (which) {
        case 2: v = V::add(V::ld(q + hq), V::ld(q + hq + h)); break;                                   // T2
        case 3: v = V::sub(V::add(V::ld(q + hq), V::ld(q + hq + h)), V::ld(q)); break;                 // T3
        case 4: v = V::sub(V::ld(q), V::ld(q + hq)); break;                                            // T4
        case 5: v = V::sub(V::ld(q + h), V::sub(V::add(V::ld(q + hq), V::ld(q + hq + h)), V::ld(q))); break;  // T5
        case 10: v = V::sub(V::ld(q + h), V::ld(q)); break;                                            // S2
        case 11: v = V::sub(V::ld(q + hq + h), V::sub(V::ld(q + h), V::ld(q))); break;                 // S3
        case 12: v = V::sub(V::ld(q + hq + h), V::ld(q + h)); break;                                   // S4
        default: v = V::sub(V::sub(V::ld(q + hq + h), V::sub(V::ld(q + h), V::ld(q))), V::ld(q + hq)); break;  // S6
        }
        V::st(O + int64_t(r) * ldo + c, v);
    }
}

// ---------------------------------------------------------------------------------------
// DFS fold of Q_j into C (Algorithm 1: "locally compute contribution of Q_i to C"), the flat
// form of the U chain:  C11 = Q0+Q1, C12 = Q0+Q3+Q2+Q5, C21 = Q0+Q3+Q4-Q6, C22 = Q0+Q3+Q4+Q2.
// Q0 writes all four quadrants (first touch), later Q_j read-modify-write theirs.
// ---------------------------------------------------------------------------------------
template <int VEC>
__global__ void __launch_bounds__(TX *TY) accumulate_kernel(const Node *__restrict__ parents,
                                                            const Node *__restrict__ children, Bases bases, int h,
                                                            int j, int item0, int peel)
{
    using V = Vec<VEC>;
    using T = typename V::type;
    const int par = item0 + blockIdx.z;
    const int c = (blockIdx.x * TX + threadIdx.x) * VEC;
    if (c >= h) return;
    const Operand qq = children[par].c, cc = parents[par].c;
    const double *Q = resolve(bases, qq);
    double *C = resolve(bases, cc);
    const int64_t ldq = qq.ld, ldc = cc.ld, hq = int64_t(h) * ldc;
    const int r0 = blockIdx.y * TILE_ROWS + threadIdx.y;
#pragma unroll
    for (int i = 0; i < ROWS_PER_THREAD; ++i) {
        const int r = r0 + i * TY;
        if (r >= h) continue;
        const T q = V::ld(Q + int64_t(r) * ldq + c);
        double *o = C + int64_t(r) * ldc + c;
        double *c11 = o, *c12 = o + h, *c21 = o + hq, *c22 = o + hq + h;
        switch (j) {
        case 0:
            if (peel) {     // odd parent: the first touch also carries the rank-one term of the peeled split
                const Operand pa = parents[par].a, pb = parents[par].b;
                const double *acol = resolve(bases, pa) + 2 * h;
                const double *brow = resolve(bases, pb) + int64_t(2 * h) * pb.ld + c;
                const double a0 = acol[int64_t(r) * pa.ld], a1 = acol[int64_t(r + h) * pa.ld];
                const T b0 = V::ldk(brow), b1 = V::ldk(brow + h);
                V::st(c11, V::fma1(a0, b0, q)); V::st(c12, V::fma1(a0, b1, q));
                V::st(c21, V::fma1(a1, b0, q)); V::st(c22, V::fma1(a1, b1, q));
            } else {
                V::st(c11, q); V::st(c12, q); V::st(c21, q); V::st(c22, q);
            }
            break;
        case 1: V::st(c11, V::add(V::ldk(c11), q)); break;
        case 2: V::st(c12, V::add(V::ldk(c12), q)); V::st(c22, V::add(V::ldk(c22), q)); break;
        case 3: V::st(c12, V::add(V::ldk(c12), q)); V::st(c21, V::add(V::ldk(c21), q));
                V::st(c22, V::add(V::ldk(c22), q)); break;
        case 4: V::st(c21, V::add(V::ldk(c21), q)); V::st(c22, V::add(V::ldk(c22), q)); break;
        case 5: V::st(c12, V::add(V::ldk(c12), q)); break;
        default: V::st(c21, V::sub(V::ldk(c21), q)); break;
        }
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
template <int VEC>
__global__ void __launch_bounds__(TX *TY) recombine2_kernel(const Node *__restrict__ parents, Bases bases, Regions2 reg,
                                                            int q, int item0, int peel)
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
                V::st(o, c11);
                V::st(o + h, c12);
                V::st(o + h * ldc, c21);
                V::st(o + h * ldc + h, c22);
            }
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
// Both read one operand in full once; summation order is fixed (bit-reproducible).

// Columns [c0, c0 + nc) of C for rows [0, rows): each warp owns 4 rows, lanes stride over k; the nc
// columns of B are staged through shared memory in chunks of TC_CHUNK rows.
constexpr int TC_ROWS = 32, TC_CHUNK = 512;
template <int NC>
__global__ void __launch_bounds__(256) thin_cols_kernel(const Node *__restrict__ nodes, Bases bases, int K, int rows,
                                                        int c0, int nc, int item0)
{
    __shared__ double bs[NC][TC_CHUNK];
    const Node nd = nodes[item0 + blockIdx.y];
    const double *A = resolve(bases, nd.a), *B = resolve(bases, nd.b);
    double *C = resolve(bases, nd.c);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rbase = blockIdx.x * TC_ROWS + warp * 4;
    double acc[4][NC];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int t = 0; t < NC; ++t) acc[i][t] = 0.0;
    for (int k0 = 0; k0 < K; k0 += TC_CHUNK) {
        const int kn = min(TC_CHUNK, K - k0);
        __syncthreads();
        for (int e = threadIdx.x; e < kn * NC; e += 256) {
            const int k = e / NC, t = e % NC;
            bs[t][k] = t < nc ? B[int64_t(k0 + k) * nd.b.ld + c0 + t] : 0.0;
        }
        __syncthreads();
        // k outer, the warp's 4 rows inner: the staged B values are read from shared memory once per k
        const double *a0 = A + int64_t(min(rbase, rows - 1)) * nd.a.ld + k0;
        const int64_t lda = nd.a.ld;
        const int nrow = min(4, rows - rbase);
        int k = lane;
        for (; k + 32 < kn; k += 64) {              // two k per lane and pass: eight loads of A in flight
            double av[2][4];
#pragma unroll
            for (int u = 0; u < 2; ++u)
#pragma unroll
                for (int i = 0; i < 4; ++i) av[u][i] = i < nrow ? a0[int64_t(i) * lda + k + 32 * u] : 0.0;
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                double bv[NC];
#pragma unroll
                for (int t = 0; t < NC; ++t) bv[t] = bs[t][k + 32 * u];
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int t = 0; t < NC; ++t) acc[i][t] = fma(av[u][i], bv[t], acc[i][t]);
            }
        }
        for (; k < kn; k += 32) {
            double bv[NC];
#pragma unroll
            for (int t = 0; t < NC; ++t) bv[t] = bs[t][k];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (i < nrow) {
                    const double av = a0[int64_t(i) * lda + k];
#pragma unroll
                    for (int t = 0; t < NC; ++t) acc[i][t] = fma(av, bv[t], acc[i][t]);
                }
            }
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = rbase + i;
#pragma unroll
        for (int t = 0; t < NC; ++t) {
            double v = acc[i][t];
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
            if (lane == 0 && r < rows && t < nc) C[int64_t(r) * nd.c.ld + c0 + t] = v;
        }
    }
}

// Rows [r0, r0 + nr) of C for columns [0, cols): a thread owns two adjacent columns and one of
// TR_SLICES interleaved pairs of k; the nr rows of A are staged through shared memory in chunks (read
// back as broadcast 16-byte pairs), and the slices are summed through shared memory in a fixed order.
constexpr int TR_COLS = 64, TR_SLICES = 8, TR_CHUNK = 512;
template <int NR>
__global__ void __launch_bounds__((TR_COLS / 2) * TR_SLICES) thin_rows_kernel(const Node *__restrict__ nodes, Bases bases,
                                                                              int K, int cols, int r0, int nr, int item0)
{
    // one buffer, used first for the staged rows of A and, after the k loop, for the slice sums
    constexpr int AS_WORDS = NR * TR_CHUNK, PART_WORDS = TR_SLICES * NR * (TR_COLS + 2);
    __shared__ __align__(16) double buf[AS_WORDS > PART_WORDS ? AS_WORDS : PART_WORDS];
    double(*as)[TR_CHUNK] = reinterpret_cast<double(*)[TR_CHUNK]>(buf);
    double(*part)[NR][TR_COLS + 2] = reinterpret_cast<double(*)[NR][TR_COLS + 2]>(buf);
    const Node nd = nodes[item0 + blockIdx.y];
    const double *A = resolve(bases, nd.a), *B = resolve(bases, nd.b);
    double *C = resolve(bases, nd.c);
    const int tid = threadIdx.y * (TR_COLS / 2) + threadIdx.x;
    const int c = blockIdx.x * TR_COLS + 2 * threadIdx.x;
    const bool c0ok = c < cols, c1ok = c + 1 < cols;
    const int64_t ldb = nd.b.ld, lda = nd.a.ld;
    const double *b = B + (c0ok ? c : 0);
    const int c1 = c1ok ? 1 : 0;
    double acc[NR][2];
#pragma unroll
    for (int t = 0; t < NR; ++t) acc[t][0] = acc[t][1] = 0.0;
    for (int k0 = 0; k0 < K; k0 += TR_CHUNK) {
        const int kn = min(TR_CHUNK, K - k0);
        __syncthreads();
        for (int e = tid; e < NR * TR_CHUNK; e += (TR_COLS / 2) * TR_SLICES) {
            const int t = e / TR_CHUNK, k = e % TR_CHUNK;
            as[t][k] = (t < nr && k < kn) ? A[int64_t(r0 + t) * lda + k0 + k] : 0.0;
        }
        __syncthreads();
        if (c0ok) {
            // slice s owns k = 2 s, 2 s + 1, then + 2 TR_SLICES, ...; entries past kn are zero in `as`
            for (int k = 2 * threadIdx.y; k < kn; k += 2 * TR_SLICES) {
                const double *bk = b + int64_t(k0 + k) * ldb;
                const bool k1ok = k + 1 < kn;
                const double b00 = bk[0], b01 = bk[c1];
                const double b10 = k1ok ? bk[ldb] : 0.0, b11 = k1ok ? bk[ldb + c1] : 0.0;
#pragma unroll
                for (int t = 0; t < NR; ++t) {
                    const double2 a2 = *reinterpret_cast<const double2 *>(&as[t][k]);
                    acc[t][0] = fma(a2.x, b00, acc[t][0]);
                    acc[t][1] = fma(a2.x, b01, acc[t][1]);
                    acc[t][0] = fma(a2.y, b10, acc[t][0]);
                    acc[t][1] = fma(a2.y, b11, acc[t][1]);
                }
            }
        }
    }
    __syncthreads();    // everyone is done reading the staged rows
#pragma unroll
    for (int t = 0; t < NR; ++t) {
        part[threadIdx.y][t][2 * threadIdx.x] = acc[t][0];
        part[threadIdx.y][t][2 * threadIdx.x + 1] = acc[t][1];
    }
    __syncthreads();
    if (threadIdx.y == 0 && c0ok) {
#pragma unroll
        for (int t = 0; t < NR; ++t) {
            double v0 = 0.0, v1 = 0.0;
#pragma unroll
            for (int i = 0; i < TR_SLICES; ++i) {
                v0 += part[i][t][2 * threadIdx.x];
                v1 += part[i][t][2 * threadIdx.x + 1];
            }
            if (t < nr) {
                C[int64_t(r0 + t) * nd.c.ld + c] = v0;
                if (c1ok) C[int64_t(r0 + t) * nd.c.ld + c + 1] = v1;
            }
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
    case OP_PEEL: return (op.peel_fused ? 2 : 3) * chunks(op.count);
    case OP_GEMM: {
        const int rem = gemm_thin_remainder(op.m), bulk = int(op.m) - rem;
        int tiled = 0;
        if (bulk > 0) {
            GemmRegion regions[4];
            tiled = gemm_regions(bulk, op.count, kNominalSMs, regions);
        }
        return tiled + (rem ? chunks(op.count) * (bulk > 0 ? 2 : 1) : 0);
    }
    case OP_FORM2: return chunks(op.count * 2);
    case OP_RECOMBINE2: return chunks(op.count);
    case OP_FORM3: return chunks(op.count * 2);
    case OP_RECOMBINE3: return chunks(op.count);
    case OP_FUSED_STEP: return chunks(op.count);
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

cudaError_t launch_recombine(const Node *tab, const Launch &op, const Bases &bases, bool vec, cudaStream_t stream,
                             int *launched)
{
    const dim3 block(TX, TY);
    const int64_t total = op.count;
    FOR_CHUNKS(total) {
        const int v = vec ? 2 : 1;
        const dim3 grid = tile_grid(op.h, v, zn);
        const Node *par = tab + op.parent_tab, *kid = tab + op.child_tab;
        if (small_grid(grid)) {
            const dim3 g1(grid.x, unsigned((op.h + TY - 1) / TY), grid.z);
            if (vec) recombine_bfs_kernel<2, 1><<<g1, block, 0, stream>>>(par, kid, bases, int(op.h), int(item0), op.peel_fused);
            else recombine_bfs_kernel<1, 1><<<g1, block, 0, stream>>>(par, kid, bases, int(op.h), int(item0), op.peel_fused);
        } else {
            if (vec) recombine_bfs_kernel<2, ROWS_PER_THREAD><<<grid, block, 0, stream>>>(par, kid, bases, int(op.h), int(item0), op.peel_fused);
            else recombine_bfs_kernel<1, ROWS_PER_THREAD><<<grid, block, 0, stream>>>(par, kid, bases, int(op.h), int(item0), op.peel_fused);
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

cudaError_t launch_recombine2(const Node *tab, const Launch &op, const Bases &bases, bool vec, cudaStream_t stream,
                              int *launched)
{
    const dim3 block(TX, TY);
    const int64_t total = op.count, q = op.h / 2;
    FOR_CHUNKS(total) {
        if (vec)
            recombine2_kernel<2><<<tile_grid(q, 2, zn), block, 0, stream>>>(tab + op.parent_tab, bases, op.reg, int(q),
                                                                           int(item0), op.peel_fused);
        else
            recombine2_kernel<1><<<tile_grid(q, 1, zn), block, 0, stream>>>(tab + op.parent_tab, bases, op.reg, int(q),
                                                                           int(item0), op.peel_fused);
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
                                                                            bases, int(op.h), j, sides, int(item0));
        else
            form_one_kernel<1><<<tile_grid(op.h, 1, zn), block, 0, stream>>>(tab + op.parent_tab, tab + op.child_tab,
                                                                            bases, int(op.h), j, sides, int(item0));
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
        const dim3 grid((rows + TC_ROWS - 1) / TC_ROWS, unsigned(zn));
        if (nc <= 1) thin_cols_kernel<1><<<grid, 256, 0, stream>>>(nodes, bases, K, rows, c0, nc, int(item0));
        else if (nc <= 2) thin_cols_kernel<2><<<grid, 256, 0, stream>>>(nodes, bases, K, rows, c0, nc, int(item0));
        else if (nc <= 4) thin_cols_kernel<4><<<grid, 256, 0, stream>>>(nodes, bases, K, rows, c0, nc, int(item0));
        else thin_cols_kernel<8><<<grid, 256, 0, stream>>>(nodes, bases, K, rows, c0, nc, int(item0));
        ++*launched;
    }
    return cudaGetLastError();
}

cudaError_t launch_thin_rows(const Node *nodes, const Bases &bases, int K, int cols, int r0, int nr, int64_t count,
                             cudaStream_t stream, int *launched)
{
    const int64_t total = count;
    FOR_CHUNKS(total) {
        const dim3 grid((cols + TR_COLS - 1) / TR_COLS, unsigned(zn)), block(TR_COLS / 2, TR_SLICES);
        if (nr <= 1) thin_rows_kernel<1><<<grid, block, 0, stream>>>(nodes, bases, K, cols, r0, nr, int(item0));
        else if (nr <= 2) thin_rows_kernel<2><<<grid, block, 0, stream>>>(nodes, bases, K, cols, r0, nr, int(item0));
        else if (nr <= 4) thin_rows_kernel<4><<<grid, block, 0, stream>>>(nodes, bases, K, cols, r0, nr, int(item0));
        else thin_rows_kernel<8><<<grid, block, 0, stream>>>(nodes, bases, K, cols, r0, nr, int(item0));
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
    cudaError_t err = launch_thin_cols(nodes, bases, m, m, e, 1, op.count, stream, launched);   // last column, all rows
    if (err != cudaSuccess) return err;
    return launch_thin_rows(nodes, bases, m, e, e, 1, op.count, stream, launched);              // last row, other columns
}

}  // namespace strassen
