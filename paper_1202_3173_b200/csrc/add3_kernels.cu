// Three consecutive BFS levels of one Strassen-Winograd recursion (Appendix A, Algorithm 1)
// formed by one streaming pass and recombined by another.
//
// A parent of size m = 2h = 8q is seen as an 8 x 8 lattice of q x q blocks; the thread at (r, c)
// owns the 64 parent elements (a q + r, b q + c).  Formation descends child by child: the
// child's operand at its 4 x 4 lattice positions, its children's operands at 2 x 2 positions,
// and the four sums of each of those; every sum is written exactly where the single-level pass
// would have put it, so that the views the deeper operands are made of stay valid.  Only the
// parent is read: per side 64 q^2 words in, instead of the 64 + 112 + 196 q^2 that three passes
// read.  Recombination runs the U-chain of Appendix A at the three levels with the intermediate
// products in registers: 343 q^2 words in, 64 q^2 out.  Both use the same operations in the same
// order as the single-level kernels, so results are bit-identical.
#include "kernels.h"
#include "fold.cuh"

namespace strassen {

namespace {

constexpr int TX3 = 64, TY3 = 4;

__device__ __forceinline__ double *resolve3(const Bases &bases, const Operand &x) { return base_ptr(bases, x.base) + x.off; }

// Operand of sub-problem j on one side, from the four quadrant values of the node's own operand:
//   A side: T0 = A11, T1 = A12, T2 = A21 + A22, T3 = T2 - A11, T4 = A11 - A21, T5 = A12 - T3, T6 = A22
//   B side: S0 = B11, S1 = B21, S2 = B12 - B11, S3 = B22 - S2, S4 = B22 - B12, S5 = B22, S6 = S3 - B21
template <int SIDE> __device__ __forceinline__ double operand_of(int j, double x11, double x12, double x21, double x22)
{
    if (SIDE == 0) {
        switch (j) {
        case 0: return x11;
        case 1: return x12;
        case 2: return x21 + x22;
        case 3: return (x21 + x22) - x11;
        case 4: return x11 - x21;
        case 5: return x12 - ((x21 + x22) - x11);
        default: return x22;
        }
    } else {
        switch (j) {
        case 0: return x11;
        case 1: return x21;
        case 2: return x12 - x11;
        case 3: return x22 - (x12 - x11);
        case 4: return x22 - x12;
        case 5: return x22;
        default: return (x22 - (x12 - x11)) - x21;
        }
    }
}
// Workspace slot of the sum that sub-problem j uses on this side, or -1 where the operand is a plain quadrant.
template <int SIDE> __device__ __forceinline__ constexpr int slot_of(int j)
{
    return SIDE == 0 ? (j >= 2 && j <= 5 ? j - 2 : -1) : (j >= 2 && j <= 4 ? j - 2 : j == 6 ? 3 : -1);
}
// Below the level that writes them, the sums are read only as the quadrant operands X11, X12, X22 (A side)
// or X11, X21, X22 (B side): the remaining quadrant is never read and is not written.
template <int SIDE> __device__ __forceinline__ constexpr bool quadrant_is_read(bool lower, bool right)
{
    return SIDE == 0 ? !(lower && !right) : !(!lower && right);
}

template <int SIDE>
__device__ __forceinline__ void form3_side(const double *__restrict__ X, int64_t ld, double *child, double *grand,
                                           double *great, const Regions2 &reg, const Regions3 &reg3, int q, int r, int c)
{
    double xv[8][8];
#pragma unroll
    for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int b = 0; b < 8; ++b) xv[a][b] = __ldcs(X + (int64_t(a) * q + r) * ld + b * q + c);
    const int64_t cld = reg.child_ld, gld = reg.grand_ld, ggld = reg3.great_ld;
#pragma unroll
    for (int j1 = 0; j1 < 7; ++j1) {
        double y1[4][4];    // operand of child j1 at its 4 x 4 lattice positions
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int v = 0; v < 4; ++v)
                y1[u][v] = operand_of<SIDE>(j1, xv[u][v], xv[u][4 + v], xv[4 + u][v], xv[4 + u][4 + v]);
        if (slot_of<SIDE>(j1) >= 0) {
            double *o = child + slot_of<SIDE>(j1) * reg.child_mat;
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int v = 0; v < 4; ++v)
                    if (quadrant_is_read<SIDE>(u >= 2, v >= 2)) o[(int64_t(u) * q + r) * cld + v * q + c] = y1[u][v];
        }
#pragma unroll
        for (int j2 = 0; j2 < 7; ++j2) {
            double y2[2][2];    // operand of grandchild (j1, j2) at its 2 x 2 lattice positions
#pragma unroll
            for (int u = 0; u < 2; ++u)
#pragma unroll
                for (int v = 0; v < 2; ++v)
                    y2[u][v] = operand_of<SIDE>(j2, y1[u][v], y1[u][2 + v], y1[2 + u][v], y1[2 + u][2 + v]);
            if (slot_of<SIDE>(j2) >= 0) {
                double *o = grand + (int64_t(j1) * 4 + slot_of<SIDE>(j2)) * reg.grand_mat;
#pragma unroll
                for (int u = 0; u < 2; ++u)
#pragma unroll
                    for (int v = 0; v < 2; ++v)
                        if (quadrant_is_read<SIDE>(u == 1, v == 1)) o[(int64_t(u) * q + r) * gld + v * q + c] = y2[u][v];
            }
            // the four sums of grandchild (j1, j2): operands of its own children
            double *o = great + (int64_t(j1) * 7 + j2) * 4 * reg3.great_mat + int64_t(r) * ggld + c;
#pragma unroll
            for (int j3 = 0; j3 < 7; ++j3)
                if (slot_of<SIDE>(j3) >= 0)
                    o[slot_of<SIDE>(j3) * reg3.great_mat] = operand_of<SIDE>(j3, y2[0][0], y2[0][1], y2[1][0], y2[1][1]);
        }
    }
}

__global__ void __launch_bounds__(TX3 *TY3) form3_kernel(const Node *__restrict__ parents, Bases bases, Regions2 reg,
                                                         Regions3 reg3, int q, int item0)
{
    const int item = item0 + blockIdx.z;
    const int par = item >> 1, side = item & 1;
    const int c = blockIdx.x * TX3 + threadIdx.x, r = blockIdx.y * TY3 + threadIdx.y;
    if (c >= q || r >= q) return;
    const Operand x = side ? parents[par].b : parents[par].a;
    double *ws = bases.p[BASE_WS];
    double *child = ws + (side ? reg.child_s : reg.child_t) + int64_t(par) * 4 * reg.child_mat;
    double *grand = ws + (side ? reg.grand_s : reg.grand_t) + int64_t(par) * 28 * reg.grand_mat;
    double *great = ws + (side ? reg3.great_s : reg3.great_t) + int64_t(par) * 196 * reg3.great_mat;
    if (side == 0) form3_side<0>(resolve3(bases, x), x.ld, child, grand, great, reg, reg3, q, r, c);
    else form3_side<1>(resolve3(bases, x), x.ld, child, grand, great, reg, reg3, q, r, c);
}

// U-chain of Appendix A over blocks of N x N lattice positions, in an order that keeps at most three
// blocks alive: U1 = Q0 + Q3, U2 = U1 + Q4, U3 = U1 + Q2; C11 = Q0 + Q1, C12 = U3 + Q5, C21 = U2 - Q6,
// C22 = U2 + Q2.  `product(j, block)` yields Q_j; `emit(quadrant, block)` consumes one quadrant of the
// result (0 = C11, 1 = C12, 2 = C21, 3 = C22).
template <int N, class Product, class Emit> __device__ __forceinline__ void u_chain(Product product, Emit emit)
{
    double p[N][N], t[N][N], u[N][N];
    auto combine = [](double (&d)[N][N], const double (&x)[N][N], const double (&y)[N][N], bool minus) {
#pragma unroll
        for (int i = 0; i < N; ++i)
#pragma unroll
            for (int k = 0; k < N; ++k) d[i][k] = minus ? x[i][k] - y[i][k] : x[i][k] + y[i][k];
    };
    double out[N][N];
    product(0, p);
    product(1, t);
    combine(out, p, t, false);      // C11 = Q0 + Q1
    emit(0, out);
    product(3, t);
    combine(p, p, t, false);        // U1 = Q0 + Q3
    product(4, t);
    combine(u, p, t, false);        // U2 = U1 + Q4
    product(6, t);
    combine(out, u, t, true);       // C21 = U2 - Q6
    emit(2, out);
    product(2, t);
    combine(out, u, t, false);      // C22 = U2 + Q2
    emit(3, out);
    combine(p, p, t, false);        // U3 = U1 + Q2
    product(5, t);
    combine(out, p, t, false);      // C12 = U3 + Q5
    emit(1, out);
}

template <bool FOLD>
__global__ void __launch_bounds__(TX3 *TY3) recombine3_kernel(const Node *__restrict__ parents, Bases bases, Regions3 reg3,
                                                              int q, int item0, int peel, const Node *__restrict__ dfs_parents,
                                                              int fold, int fold_peel)
{
    // FOLD (fold != 0): the parents are the sub-problems j = fold - 1 of a DFS step one level up; their products are folded
    // into the C quadrants of those DFS parents instead of being written
    // last parent first: its products are the ones the preceding kernel wrote last, so they are still in L2
    const int par = item0 + (gridDim.z - 1 - blockIdx.z);
    const int c = blockIdx.x * TX3 + threadIdx.x, r = blockIdx.y * TY3 + threadIdx.y;
    if (c >= q || r >= q) return;
    const Operand cc = parents[par].c;
    double *C = resolve3(bases, cc);
    const int64_t ldc = cc.ld;
    const double *great = bases.p[BASE_WS] + reg3.great_q + int64_t(par) * 343 * reg3.great_mat + int64_t(r) * reg3.great_ld + c;
    const int64_t mat = reg3.great_mat;
    FoldTarget ft{};
    if (FOLD) ft = fold_target(dfs_parents[par], bases, 8 * q, fold - 1, fold_peel);
    // peel != 0: parent of odd size 8q + 1; every entry also gets A[row][8q] * B[8q][col], the rank-one
    // term of the peeled split
    const double *acol = nullptr, *brow = nullptr;
    int64_t lda = 0;
    if (peel) {
        const Operand pa = parents[par].a, pb = parents[par].b;
        acol = resolve3(bases, pa) + 8 * q;
        lda = pa.ld;
        brow = resolve3(bases, pb) + int64_t(8 * q) * pb.ld + c;
    }
    u_chain<4>(
        [&](int j1, double (&z1)[4][4]) {       // product of child j1 at its 4 x 4 lattice positions
            u_chain<2>(
                [&](int j2, double (&z2)[2][2]) {       // product of grandchild (j1, j2) at 2 x 2 positions
                    const double *g = great + (int64_t(j1) * 7 + j2) * 7 * mat;
                    double k[7];
#pragma unroll
                    for (int t = 0; t < 7; ++t) k[t] = __ldcs(g + t * mat);
                    const double u1 = k[0] + k[3], u2 = u1 + k[4], u3 = u1 + k[2];
                    z2[0][0] = k[0] + k[1];
                    z2[0][1] = u3 + k[5];
                    z2[1][0] = u2 - k[6];
                    z2[1][1] = u2 + k[2];
                },
                [&](int quad, const double (&b)[2][2]) {
#pragma unroll
                    for (int u = 0; u < 2; ++u)
#pragma unroll
                        for (int v = 0; v < 2; ++v) z1[(quad >> 1) * 2 + u][(quad & 1) * 2 + v] = b[u][v];
                });
        },
        [&](int quad, const double (&b)[4][4]) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int a = (quad >> 1) * 4 + u;
                const double av = peel ? acol[(int64_t(a) * q + r) * lda] : 0.0;
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    const int bb = (quad & 1) * 4 + v;
                    double val = b[u][v];
                    if (peel) val = fma(av, brow[bb * q], val);
                    if (FOLD) fold_emit<1>(ft, a * q + r, bb * q + c, val);
                    else C[(int64_t(a) * q + r) * ldc + bb * q + c] = val;
                }
            }
        });
}

}  // namespace

#define FOR_CHUNKS3(total)                                                    \
    for (int64_t item0 = 0, zn; item0 < (total); item0 += kMaxItemsPerLaunch) \
        if ((zn = ((total) - item0 < kMaxItemsPerLaunch ? (total) - item0 : kMaxItemsPerLaunch)), true)

cudaError_t launch_form3(const Node *tab, const Launch &op, const Bases &bases, cudaStream_t stream, int *launched)
{
    const dim3 block(TX3, TY3);
    const int64_t total = op.count * 2, q = op.h / 4;
    FOR_CHUNKS3(total) {
        const dim3 grid(unsigned((q + TX3 - 1) / TX3), unsigned((q + TY3 - 1) / TY3), unsigned(zn));
        form3_kernel<<<grid, block, 0, stream>>>(tab + op.parent_tab, bases, op.reg, op.reg3, int(q), int(item0));
        ++*launched;
    }
    return cudaGetLastError();
}

cudaError_t launch_recombine3(const Node *tab, const Launch &op, const Bases &bases, cudaStream_t stream, int *launched)
{
    const dim3 block(TX3, TY3);
    const int64_t total = op.count, q = op.h / 4;
    FOR_CHUNKS3(total) {
        const dim3 grid(unsigned((q + TX3 - 1) / TX3), unsigned((q + TY3 - 1) / TY3), unsigned(zn));
        if (op.fold)
            recombine3_kernel<true><<<grid, block, 0, stream>>>(tab + op.parent_tab, bases, op.reg3, int(q), int(item0), op.peel_fused,
                                                                tab + op.fold_tab, op.fold, op.fold_peel);
        else
            recombine3_kernel<false><<<grid, block, 0, stream>>>(tab + op.parent_tab, bases, op.reg3, int(q), int(item0), op.peel_fused,
                                                                 nullptr, 0, 0);
        ++*launched;
    }
    return cudaGetLastError();
}

}  // namespace strassen
