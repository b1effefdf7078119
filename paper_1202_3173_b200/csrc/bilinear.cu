// The one streaming kernel of the generic <n0, n0, n0; q> bilinear schemes (Section 6.6): one output matrix per
// parent as a linear combination, with small integer coefficients, of up to 16 input matrices --
//   * an operand T_j (S_j) of a sub-problem from the n0 x n0 blocks of the parent's A (B),
//   * a block of the parent's C from the products Q_j of its sub-problems (BFS step), or the contribution of one
//     Q_j added to it (DFS step).
// HBM-bound: every term is read once per output element.  Terms are added in table order, each as coefficient
// times value (coefficients +-1 are exact), so results are reproducible.
#include "bilinear.h"
#include "kernels.h"

namespace strassen {

namespace {

constexpr int LX = 64, LY = 4;

// NT = most terms this instantiation adds (4, 8 or 16), ROWS = rows per thread (4, 2, 1): all ROWS x NT loads of a
// thread are issued before the first addition, so that enough of them are in flight to cover the memory latency.
template <int VEC, int NT, int ROWS>
__global__ void __launch_bounds__(LX *LY) lincomb_kernel(const Node *__restrict__ parents, const Node *__restrict__ children, Bases bases,
                                                         LinComb lc, int hh, int item0)
{
    const int par = item0 + blockIdx.z;
    const int c = (blockIdx.x * LX + threadIdx.x) * VEC;
    if (c >= hh) return;
    const Node nd = parents[par];
    const Node *kids = children + (long long)par * lc.children;
    const double *src[NT];
    long long lds[NT];
    double *out;
    long long ldo;
    if (lc.mode == 2) {
#pragma unroll
        for (int i = 0; i < NT; ++i) {
            const Operand x = kids[i < lc.nterms ? lc.src[i] : 0].c;
            src[i] = base_ptr(bases, x.base) + x.off;
            lds[i] = x.ld;
        }
        out = base_ptr(bases, nd.c.base) + nd.c.off + (long long)(lc.out / lc.n0) * hh * nd.c.ld + (long long)(lc.out % lc.n0) * hh;
        ldo = nd.c.ld;
    } else {
        const Operand x = lc.mode ? nd.b : nd.a;
        const double *X = base_ptr(bases, x.base) + x.off;
#pragma unroll
        for (int i = 0; i < NT; ++i) {
            const int b = i < lc.nterms ? lc.src[i] : 0;
            src[i] = X + (long long)(b / lc.n0) * hh * x.ld + (long long)(b % lc.n0) * hh;
            lds[i] = x.ld;
        }
        const Operand y = lc.mode ? kids[lc.out].b : kids[lc.out].a;
        out = base_ptr(bases, y.base) + y.off;
        ldo = y.ld;
    }
    const int r0 = blockIdx.y * (LY * ROWS) + threadIdx.y;
    double v[ROWS][NT][VEC], prev[ROWS][VEC];
#pragma unroll
    for (int k = 0; k < ROWS; ++k) {
        const int r = r0 + k * LY;
#pragma unroll
        for (int i = 0; i < NT; ++i) {
            const bool on = r < hh && i < lc.nterms;
            const double *s = src[i] + (long long)r * lds[i] + c;
            if (VEC == 2) {
                const double2 x = on ? __ldcs(reinterpret_cast<const double2 *>(s)) : make_double2(0.0, 0.0);
                v[k][i][0] = x.x;
                v[k][i][VEC - 1] = x.y;
            } else {
                v[k][i][0] = on ? __ldcs(s) : 0.0;
            }
        }
#pragma unroll
        for (int e = 0; e < VEC; ++e) prev[k][e] = (lc.accumulate && r < hh) ? out[(long long)r * ldo + c + e] : 0.0;
    }
#pragma unroll
    for (int k = 0; k < ROWS; ++k) {
        const int r = r0 + k * LY;
        if (r >= hh) continue;
        double acc[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
            // terms in table order; the first one starts the sum unless the block already holds one
            acc[e] = lc.accumulate ? prev[k][e] + double(lc.coef[0]) * v[k][0][e] : double(lc.coef[0]) * v[k][0][e];
#pragma unroll
            for (int i = 1; i < NT; ++i)
                if (i < lc.nterms) acc[e] = acc[e] + double(lc.coef[i]) * v[k][i][e];
        }
        if (VEC == 2) *reinterpret_cast<double2 *>(out + (long long)r * ldo + c) = make_double2(acc[0], acc[VEC - 1]);
        else out[(long long)r * ldo + c] = acc[0];
    }
}

template <int VEC, int NT, int ROWS>
void launch_lincomb_as(const Node *tab, const Launch &op, const LinComb &lc, const Bases &bases, int64_t item0, int64_t zn, cudaStream_t stream)
{
    const int hh = int(op.h);
    const dim3 block(LX, LY), grid(unsigned((hh + LX * VEC - 1) / (LX * VEC)), unsigned((hh + LY * ROWS - 1) / (LY * ROWS)), unsigned(zn));
    lincomb_kernel<VEC, NT, ROWS><<<grid, block, 0, stream>>>(tab + op.parent_tab, tab + op.child_tab, bases, lc, hh, int(item0));
}

}  // namespace

cudaError_t launch_lincomb(const Node *tab, const Launch &op, const LinComb &lc, const Bases &bases, bool vec, cudaStream_t stream,
                           int *launched)
{
    for (int64_t item0 = 0; item0 < op.count; item0 += kMaxItemsPerLaunch) {
        const int64_t zn = op.count - item0 < kMaxItemsPerLaunch ? op.count - item0 : kMaxItemsPerLaunch;
        if (lc.nterms <= 4) {
            if (vec) launch_lincomb_as<2, 4, 4>(tab, op, lc, bases, item0, zn, stream);
            else launch_lincomb_as<1, 4, 4>(tab, op, lc, bases, item0, zn, stream);
        } else if (lc.nterms <= 8) {
            if (vec) launch_lincomb_as<2, 8, 2>(tab, op, lc, bases, item0, zn, stream);
            else launch_lincomb_as<1, 8, 2>(tab, op, lc, bases, item0, zn, stream);
        } else {
            if (vec) launch_lincomb_as<2, 16, 1>(tab, op, lc, bases, item0, zn, stream);
            else launch_lincomb_as<1, 16, 1>(tab, op, lc, bases, item0, zn, stream);
        }
        ++*launched;
    }
    return cudaGetLastError();
}

}  // namespace strassen
