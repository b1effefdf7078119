// Diagonal scaling (Section 6.1): D1 C D3 = (D1 A D2)(D2^-1 B D3) with power-of-two diagonals, so that the
// scaling itself is exact.  Inside scaling (D2) balances column k of A against row k of B; outside scaling
// (D1, D3) brings the largest entry of every row of A D2 and of every column of D2^-1 B into [1, 2).  All
// kernels are HBM streaming passes over n x n matrices; exponents are kept as int32, three arrays of n per
// batch member (e1, e2, e3), zero where a scaling is switched off.
#include <climits>

#include "kernels.h"

namespace strassen {

namespace {

__device__ __forceinline__ int ilog2_abs(double m) { return m > 0.0 ? ilogb(m) : 0; }   // floor(log2 m), 0 for 0

// out[i] = sign * ilog2( max_k |X[i][k]| 2^(csign * cexp[k]) ); one warp per row.
__global__ void __launch_bounds__(256) rowmax_ilog2_kernel(const double *X, int64_t ld, int64_t stride, int n,
                                                           const int *cexp, int csign, int *out, int sign)
{
    const int b = blockIdx.y;
    const int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (row >= n) return;
    const double *x = X + b * stride + int64_t(row) * ld;
    const int *ce = cexp ? cexp + int64_t(b) * n : nullptr;
    double m = 0.0;
    int k = lane;
    for (; k + 96 < n; k += 128) {                  // four loads in flight per lane
        double v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = fabs(x[k + 32 * u]);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (ce) v[u] = scalbn(v[u], csign * ce[k + 32 * u]);
            m = fmax(m, v[u]);
        }
    }
    for (; k < n; k += 32) {
        double v = fabs(x[k]);
        if (ce) v = scalbn(v, csign * ce[k]);
        m = fmax(m, v);
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, d));
    if (lane == 0) out[int64_t(b) * n + row] = sign * ilog2_abs(m);
}

// out[j] = sign * ilog2( max_i |X[i][j]| 2^(rsign * rexp[i]) ); a CTA owns 32 columns, 32 row slices.
constexpr int CM_SLICES = 32;
__global__ void __launch_bounds__(32 * CM_SLICES) colmax_ilog2_kernel(const double *X, int64_t ld, int64_t stride, int n,
                                                           const int *rexp, int rsign, int *out, int sign)
{
    __shared__ double part[CM_SLICES][33];
    const int b = blockIdx.y;
    const int col = blockIdx.x * 32 + threadIdx.x;
    const double *x = X + b * stride;
    const int *re = rexp ? rexp + int64_t(b) * n : nullptr;
    double m = 0.0;
    if (col < n) {
        int i = threadIdx.y;
        for (; i + 3 * CM_SLICES < n; i += 4 * CM_SLICES) {      // four loads in flight per thread
            double v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) v[u] = fabs(x[int64_t(i + u * CM_SLICES) * ld + col]);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (re) v[u] = scalbn(v[u], rsign * re[i + u * CM_SLICES]);
                m = fmax(m, v[u]);
            }
        }
        for (; i < n; i += CM_SLICES) {
            double v = fabs(x[int64_t(i) * ld + col]);
            if (re) v = scalbn(v, rsign * re[i]);
            m = fmax(m, v);
        }
    }
    part[threadIdx.y][threadIdx.x] = m;
    __syncthreads();
    if (threadIdx.y == 0 && col < n) {
#pragma unroll
        for (int s = 1; s < CM_SLICES; ++s) m = fmax(m, part[s][threadIdx.x]);
        out[int64_t(b) * n + col] = sign * ilog2_abs(m);
    }
}

// e2[k] = floor((lb[k] - la[k]) / 2) in place of lb (la, lb = ilog2 of column maxima of A / row maxima of B)
__global__ void combine_inside_kernel(const int *la, int *lb_e2, int64_t count)
{
    const int64_t i = blockIdx.x * 256ll + threadIdx.x;
    if (i < count) {
        const int d = lb_e2[i] - la[i];
        lb_e2[i] = d >= 0 ? d / 2 : -((-d + 1) / 2);
    }
}

__global__ void fill_int_kernel(int *p, int64_t count, int v)
{
    const int64_t i = blockIdx.x * 256ll + threadIdx.x;
    if (i < count) p[i] = v;
}

// Y[i][j] = X[i][j] 2^(rsign rexp[i] + csign cexp[j])
__global__ void __launch_bounds__(256) scale_copy_kernel(const double *X, int64_t ldx, int64_t sx, double *Y, int64_t ldy,
                                                         int64_t sy, int n, const int *rexp, int rsign, const int *cexp,
                                                         int csign)
{
    const int b = blockIdx.z;
    const int col = blockIdx.x * 64 + threadIdx.x;
    if (col >= n) return;
    const int ec = csign * cexp[int64_t(b) * n + col];
    const int r0 = blockIdx.y * 16 + threadIdx.y;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = r0 + 4 * i;
        if (r < n)
            Y[b * sy + int64_t(r) * ldy + col] = scalbn(X[b * sx + int64_t(r) * ldx + col], rsign * rexp[int64_t(b) * n + r] + ec);
    }
}

}  // namespace

int scale_launches(const PlanDesc &d, bool in)
{
    if (!in) return 1;
    return (d.scale_inside ? 3 : 1) + (d.scale_outside ? 2 : 2) + 2;
}

// Exponents, then the scaled copies of A and B in the workspace.
cudaError_t launch_scale_in(const PlanDesc &d, const Bases &bases, cudaStream_t stream, int *launched)
{
    const int n = int(d.n);
    const int64_t cnt = d.batch * d.n;
    int *e1 = reinterpret_cast<int *>(bases.p[BASE_WS] + d.scale_exp_off), *e2 = e1 + cnt, *e3 = e2 + cnt;
    const double *A = bases.p[BASE_A], *B = bases.p[BASE_B];
    double *As = bases.p[BASE_WS] + d.scale_a_off, *Bs = bases.p[BASE_WS] + d.scale_b_off;
    const unsigned fill_grid = unsigned((cnt + 255) / 256);
    const dim3 rgrid((n + 7) / 8, unsigned(d.batch)), cgrid((n + 31) / 32, unsigned(d.batch));
    if (d.scale_inside) {
        colmax_ilog2_kernel<<<cgrid, dim3(32, CM_SLICES), 0, stream>>>(A, d.lda, d.stride_a, n, nullptr, 0, e1, 1);   // la in e1 (scratch)
        rowmax_ilog2_kernel<<<rgrid, 256, 0, stream>>>(B, d.ldb, d.stride_b, n, nullptr, 0, e2, 1);            // lb in e2
        combine_inside_kernel<<<fill_grid, 256, 0, stream>>>(e1, e2, cnt);
        *launched += 3;
    } else {
        fill_int_kernel<<<fill_grid, 256, 0, stream>>>(e2, cnt, 0);
        *launched += 1;
    }
    if (d.scale_outside) {
        rowmax_ilog2_kernel<<<rgrid, 256, 0, stream>>>(A, d.lda, d.stride_a, n, e2, 1, e1, -1);               // e1 = -ilog2 rowmax(A D2)
        colmax_ilog2_kernel<<<cgrid, dim3(32, CM_SLICES), 0, stream>>>(B, d.ldb, d.stride_b, n, e2, -1, e3, -1);       // e3 = -ilog2 colmax(D2^-1 B)
    } else {
        fill_int_kernel<<<fill_grid, 256, 0, stream>>>(e1, cnt, 0);
        fill_int_kernel<<<fill_grid, 256, 0, stream>>>(e3, cnt, 0);
    }
    *launched += 2;
    const dim3 sgrid((n + 63) / 64, (n + 15) / 16, unsigned(d.batch)), sblock(64, 4);
    scale_copy_kernel<<<sgrid, sblock, 0, stream>>>(A, d.lda, d.stride_a, As, d.scale_ld, d.scale_ld * d.n, n, e1, 1, e2, 1);
    scale_copy_kernel<<<sgrid, sblock, 0, stream>>>(B, d.ldb, d.stride_b, Bs, d.scale_ld, d.scale_ld * d.n, n, e2, -1, e3, 1);
    *launched += 2;
    return cudaGetLastError();
}

// C[i][j] *= 2^(-e1[i] - e3[j]) in place.
cudaError_t launch_scale_out(const PlanDesc &d, const Bases &bases, cudaStream_t stream, int *launched)
{
    const int n = int(d.n);
    const int64_t cnt = d.batch * d.n;
    const int *e1 = reinterpret_cast<const int *>(bases.p[BASE_WS] + d.scale_exp_off), *e3 = e1 + 2 * cnt;
    const dim3 sgrid((n + 63) / 64, (n + 15) / 16, unsigned(d.batch)), sblock(64, 4);
    scale_copy_kernel<<<sgrid, sblock, 0, stream>>>(bases.p[BASE_C], d.ldc, d.stride_c, bases.p[BASE_C], d.ldc, d.stride_c, n,
                                                    e1, -1, e3, -1);
    *launched += 1;
    return cudaGetLastError();
}

}  // namespace strassen
