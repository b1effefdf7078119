// Device helpers shared by the streaming kernels: one- and two-element accessors, and the fold of a
// sub-problem's product into the C quadrants of the DFS step above it.
#pragma once
#include "kernels.h"

namespace strassen {

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
    static __device__ __forceinline__ double ldu(const double *p) { return *p; }
    static __device__ __forceinline__ void stu(double *p, double v) { *p = v; }
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
    // two adjacent elements that need not start on a 16-byte boundary (rows of a matrix with an odd leading dimension
    // alternate between aligned and not): one 16-byte access where they do, two 8-byte ones where they do not
    static __device__ __forceinline__ double2 ldu(const double *p)
    {
        if ((reinterpret_cast<uintptr_t>(p) & 15) == 0) return *reinterpret_cast<const double2 *>(p);
        return make_double2(p[0], p[1]);
    }
    static __device__ __forceinline__ void stu(double *p, double2 v)
    {
        if ((reinterpret_cast<uintptr_t>(p) & 15) == 0) {
            *reinterpret_cast<double2 *>(p) = v;
        } else {
            p[0] = v.x;
            p[1] = v.y;
        }
    }
};

__device__ __forceinline__ double *resolve(const Bases &bases, const Operand &x) { return base_ptr(bases, x.base) + x.off; }

// ---------------------------------------------------------------------------------------
// DFS fold of Q_j into C (Algorithm 1: "locally compute contribution of Q_i to C"), the flat
// form of the U chain:  C11 = Q0+Q1, C12 = Q0+Q3+Q2+Q5, C21 = Q0+Q3+Q4-Q6, C22 = Q0+Q3+Q4+Q2.
// Q0 writes all four quadrants (first touch), later Q_j read-modify-write theirs.
// ---------------------------------------------------------------------------------------
struct FoldTarget {
    double *P;             // C of the DFS parent (size 2H, or 2H + 1 when peeled)
    const double *acol;    // odd parent, j = 0: its A[:, 2H] and B[2H, :] (the first touch also carries the rank-one
    const double *brow;    // term of the peeled split); otherwise nullptr
    long long ldp, lda;
    int H, j;
};

__device__ __forceinline__ FoldTarget fold_target(const Node &dfs_parent, const Bases &bases, int H, int j, int peel)
{
    FoldTarget f;
    f.P = resolve(bases, dfs_parent.c);
    f.ldp = dfs_parent.c.ld;
    f.H = H;
    f.j = j;
    f.acol = nullptr;
    f.brow = nullptr;
    f.lda = 0;
    if (peel && j == 0) {
        f.acol = resolve(bases, dfs_parent.a) + 2 * H;
        f.lda = dfs_parent.a.ld;
        f.brow = resolve(bases, dfs_parent.b) + (long long)(2 * H) * dfs_parent.b.ld;
    }
    return f;
}

// v = Q_j at rows R, columns C .. C + VEC - 1 of the sub-problem's product.  TOLERANT: the parent's C (and, for the
// rank-one term, its B) may sit where 16-byte accesses are not allowed although the sub-problem's own matrices allow
// them (a parent with an odd leading dimension): every access to the parent then checks its own alignment.
template <int VEC, bool TOLERANT = false>
__device__ __forceinline__ void fold_emit(const FoldTarget &f, int R, int C, typename Vec<VEC>::type v)
{
    using V = Vec<VEC>;
    using T = typename V::type;
    double *c11 = f.P + (long long)R * f.ldp + C, *c12 = c11 + f.H, *c21 = c11 + (long long)f.H * f.ldp, *c22 = c21 + f.H;
    auto ld = [](const double *p) { return TOLERANT ? V::ldu(p) : V::ldk(p); };
    auto st = [](double *p, T x) {
        if (TOLERANT) V::stu(p, x);
        else V::st(p, x);
    };
    switch (f.j) {
    case 0:
        if (f.acol) {
            const double a0 = f.acol[(long long)R * f.lda], a1 = f.acol[(long long)(R + f.H) * f.lda];
            const T b0 = ld(f.brow + C), b1 = ld(f.brow + C + f.H);
            st(c11, V::fma1(a0, b0, v)); st(c12, V::fma1(a0, b1, v));
            st(c21, V::fma1(a1, b0, v)); st(c22, V::fma1(a1, b1, v));
        } else {
            st(c11, v); st(c12, v); st(c21, v); st(c22, v);
        }
        break;
    case 1: st(c11, V::add(ld(c11), v)); break;
    case 2: st(c12, V::add(ld(c12), v)); st(c22, V::add(ld(c22), v)); break;
    case 3: st(c12, V::add(ld(c12), v)); st(c21, V::add(ld(c21), v));
            st(c22, V::add(ld(c22), v)); break;
    case 4: st(c21, V::add(ld(c21), v)); st(c22, V::add(ld(c22), v)); break;
    case 5: st(c12, V::add(ld(c12), v)); break;
    default: st(c21, V::sub(ld(c21), v)); break;
    }
}

}  // namespace strassen
