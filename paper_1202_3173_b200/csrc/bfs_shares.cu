// The two local steps of a BFS step that is spread over seven processors (Algorithm 2, BFS(A, B, C, k):
// "locally compute T_i, S_i" before the redistribution and "locally compute C from Q_i" after it), on
// one rank's share of the matrices.
//
// Data layout (Section 3.2: every processor owns the same part of each quadrant, so the additions
// need no communication).  With h = n / 2, the h rows of every quadrant are cut into seven consecutive
// blocks; rank r owns block r of each of the four quadrants.  Its share of A is stored as a
// (2 rows) x (2 h) row-major matrix: [A11_r | A12_r] on top of [A21_r | A22_r], `rows` = the size of
// block r; likewise B and C.  Forming the operands of sub-problem j on the share gives block r of T_j
// and S_j (rows x h each): the message rank r sends to rank j, n^2 / (4 P) words when 7 divides h
// (Section 3.3).  After the exchange rank j holds all seven blocks, i.e. T_j and S_j in full, multiplies
// them with the single-GPU path, and sends block r of Q_j back to rank r, which combines its seven
// blocks into its share of C.
//
// Both kernels are plain streaming passes (HBM-bound): every input element read once, every output
// written once.  The seven outputs / inputs are given as seven pointers, so the caller decides where
// each block lives (one send buffer, or a buffer per destination).
#include "strassen_b200.h"

#include <string>

#include "kernels.h"

using namespace strassen;

namespace {

struct Ptr7 {
    double *p[7];
};

constexpr int BX = 64, BY = 4;

template <int VEC> struct Acc;
template <> struct Acc<1> {
    using T = double;
    static __device__ __forceinline__ T ld(const double *p) { return __ldcs(p); }
    static __device__ __forceinline__ void st(double *p, T v) { *p = v; }
    static __device__ __forceinline__ T add(T a, T b) { return a + b; }
    static __device__ __forceinline__ T sub(T a, T b) { return a - b; }
};
template <> struct Acc<2> {
    using T = double2;
    static __device__ __forceinline__ T ld(const double *p) { return __ldcs(reinterpret_cast<const double2 *>(p)); }
    static __device__ __forceinline__ void st(double *p, T v) { *reinterpret_cast<double2 *>(p) = v; }
    static __device__ __forceinline__ T add(T a, T b) { return make_double2(a.x + b.x, a.y + b.y); }
    static __device__ __forceinline__ T sub(T a, T b) { return make_double2(a.x - b.x, a.y - b.y); }
};

// blockIdx.z = side: 0 forms block r of T_0 .. T_6 from the share of A, 1 block r of S_0 .. S_6 from the share of B
// (Appendix A):  T0 = A11  T1 = A12  T2 = A21 + A22  T3 = T2 - A11  T4 = A11 - A21  T5 = A12 - T3  T6 = A22
//                S0 = B11  S1 = B21  S2 = B12 - B11  S3 = B22 - S2  S4 = B22 - B12  S5 = B22       S6 = S3 - B21
template <int VEC>
__global__ void __launch_bounds__(BX *BY) form_shares_kernel(const double *__restrict__ A, long long lda, const double *__restrict__ B,
                                                             long long ldb, Ptr7 T, Ptr7 S, long long ldo, int rows, int h)
{
    using V = Acc<VEC>;
    using E = typename V::T;
    const int c = (blockIdx.x * BX + threadIdx.x) * VEC, r = blockIdx.y * BY + threadIdx.y;
    if (c >= h || r >= rows) return;
    const int side = blockIdx.z;
    const double *X = side ? B : A;
    const long long ld = side ? ldb : lda;
    const double *x = X + (long long)r * ld + c;
    const E x11 = V::ld(x), x12 = V::ld(x + h), x21 = V::ld(x + (long long)rows * ld), x22 = V::ld(x + (long long)rows * ld + h);
    const long long o = (long long)r * ldo + c;
    if (side == 0) {
        const E t2 = V::add(x21, x22), t3 = V::sub(t2, x11);
        V::st(T.p[0] + o, x11); V::st(T.p[1] + o, x12); V::st(T.p[2] + o, t2); V::st(T.p[3] + o, t3);
        V::st(T.p[4] + o, V::sub(x11, x21)); V::st(T.p[5] + o, V::sub(x12, t3)); V::st(T.p[6] + o, x22);
    } else {
        const E s2 = V::sub(x12, x11), s3 = V::sub(x22, s2);
        V::st(S.p[0] + o, x11); V::st(S.p[1] + o, x21); V::st(S.p[2] + o, s2); V::st(S.p[3] + o, s3);
        V::st(S.p[4] + o, V::sub(x22, x12)); V::st(S.p[5] + o, x22); V::st(S.p[6] + o, V::sub(s3, x21));
    }
}

// Block r of Q_0 .. Q_6 -> the rank's share of C:  U1 = Q0 + Q3  U2 = U1 + Q4  U3 = U1 + Q2
//   C11 = Q0 + Q1  C12 = U3 + Q5  C21 = U2 - Q6  C22 = U2 + Q2
template <int VEC>
__global__ void __launch_bounds__(BX *BY) combine_shares_kernel(Ptr7 Q, long long ldq, double *__restrict__ C, long long ldc, int rows, int h)
{
    using V = Acc<VEC>;
    using E = typename V::T;
    const int c = (blockIdx.x * BX + threadIdx.x) * VEC, r = blockIdx.y * BY + threadIdx.y;
    if (c >= h || r >= rows) return;
    const long long i = (long long)r * ldq + c;
    E q[7];
#pragma unroll
    for (int j = 0; j < 7; ++j) q[j] = V::ld(Q.p[j] + i);
    const E u1 = V::add(q[0], q[3]), u2 = V::add(u1, q[4]), u3 = V::add(u1, q[2]);
    double *o = C + (long long)r * ldc + c;
    V::st(o, V::add(q[0], q[1]));
    V::st(o + h, V::add(u3, q[5]));
    V::st(o + (long long)rows * ldc, V::sub(u2, q[6]));
    V::st(o + (long long)rows * ldc + h, V::add(u2, q[2]));
}

int shares_fail(int status, const std::string &msg)
{
    set_last_error(msg.c_str());
    return status;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
bool aligned8(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 7) == 0; }

}  // namespace

extern "C" int strassen_bfs_form_shares(int64_t rows, int64_t h, const double *A_share, int64_t lda, const double *B_share,
                                        int64_t ldb, double *const *T_out, double *const *S_out, int64_t ld_out, void *stream_v)
{
    set_last_error("");
    if (rows < 0 || h < 1 || h > (int64_t(1) << 30) || rows > h) return shares_fail(STRASSEN_INVALID_ARG, "need 0 <= rows <= h, 1 <= h <= 2^30");
    if (!A_share || !B_share || !T_out || !S_out) return shares_fail(STRASSEN_INVALID_ARG, "shares and output pointer arrays must be non-NULL");
    if (lda < 2 * h || ldb < 2 * h || ld_out < h) return shares_fail(STRASSEN_INVALID_ARG, "lda, ldb must be >= 2 h and ld_out >= h");
    Ptr7 T, S;
    bool vec = aligned16(A_share) && aligned16(B_share) && (lda % 2 == 0) && (ldb % 2 == 0) && (ld_out % 2 == 0) && (h % 2 == 0);
    for (int j = 0; j < 7; ++j) {
        T.p[j] = T_out[j];
        S.p[j] = S_out[j];
        if (!T.p[j] || !S.p[j]) return shares_fail(STRASSEN_INVALID_ARG, "an output block pointer is NULL");
        if (!aligned8(T.p[j]) || !aligned8(S.p[j])) return shares_fail(STRASSEN_MISALIGNED, "output blocks must be 8-byte aligned");
        vec = vec && aligned16(T.p[j]) && aligned16(S.p[j]);
    }
    if (!aligned8(A_share) || !aligned8(B_share)) return shares_fail(STRASSEN_MISALIGNED, "shares must be 8-byte aligned");
    if (rows == 0) return STRASSEN_OK;       // a rank whose block is empty (h < 7) has nothing to form
    if (rows > 65535 * BY) return shares_fail(STRASSEN_INVALID_ARG, "a share of more than 262140 rows is not supported");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const int v = vec ? 2 : 1;
    const dim3 grid(unsigned((h + BX * v - 1) / (BX * v)), unsigned((rows + BY - 1) / BY), 2), block(BX, BY);
    if (vec) form_shares_kernel<2><<<grid, block, 0, stream>>>(A_share, lda, B_share, ldb, T, S, ld_out, int(rows), int(h));
    else form_shares_kernel<1><<<grid, block, 0, stream>>>(A_share, lda, B_share, ldb, T, S, ld_out, int(rows), int(h));
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return shares_fail(STRASSEN_CUDA_ERROR, std::string("form_shares launch: ") + cudaGetErrorString(e));
    return STRASSEN_OK;
}

extern "C" int strassen_bfs_combine_shares(int64_t rows, int64_t h, const double *const *Q_in, int64_t ldq, double *C_share,
                                           int64_t ldc, void *stream_v)
{
    set_last_error("");
    if (rows < 0 || h < 1 || h > (int64_t(1) << 30) || rows > h) return shares_fail(STRASSEN_INVALID_ARG, "need 0 <= rows <= h, 1 <= h <= 2^30");
    if (!Q_in || !C_share) return shares_fail(STRASSEN_INVALID_ARG, "product blocks and the share of C must be non-NULL");
    if (ldq < h || ldc < 2 * h) return shares_fail(STRASSEN_INVALID_ARG, "ldq must be >= h and ldc >= 2 h");
    if (!aligned8(C_share)) return shares_fail(STRASSEN_MISALIGNED, "the share of C must be 8-byte aligned");
    Ptr7 Q;
    bool vec = aligned16(C_share) && (ldq % 2 == 0) && (ldc % 2 == 0) && (h % 2 == 0);
    for (int j = 0; j < 7; ++j) {
        Q.p[j] = const_cast<double *>(Q_in[j]);
        if (!Q.p[j]) return shares_fail(STRASSEN_INVALID_ARG, "a product block pointer is NULL");
        if (!aligned8(Q.p[j])) return shares_fail(STRASSEN_MISALIGNED, "product blocks must be 8-byte aligned");
        vec = vec && aligned16(Q.p[j]);
    }
    if (rows == 0) return STRASSEN_OK;
    if (rows > 65535 * BY) return shares_fail(STRASSEN_INVALID_ARG, "a share of more than 262140 rows is not supported");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const int v = vec ? 2 : 1;
    const dim3 grid(unsigned((h + BX * v - 1) / (BX * v)), unsigned((rows + BY - 1) / BY)), block(BX, BY);
    if (vec) combine_shares_kernel<2><<<grid, block, 0, stream>>>(Q, ldq, C_share, ldc, int(rows), int(h));
    else combine_shares_kernel<1><<<grid, block, 0, stream>>>(Q, ldq, C_share, ldc, int(rows), int(h));
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return shares_fail(STRASSEN_CUDA_ERROR, std::string("combine_shares launch: ") + cudaGetErrorString(e));
    return STRASSEN_OK;
}
