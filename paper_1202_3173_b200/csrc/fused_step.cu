// One whole Strassen-Winograd step in a single kernel (Appendix A; Algorithm 1 with its three
// "locally compute" lines collapsed): C = A.B for parents of size 2h (+1 when peeled) straight from
// the quadrants of A and B, with no operand sums, no products and no node table for the children
// ever reaching memory.
//
// A CTA owns a tile of positions (r, c) of the h x h quadrant grid and computes all seven
// products Q_0..Q_6 at those positions at once:
//   * the loader stages, per 16-deep slab, the tile's rows of the four quadrants of A and the
//     tile's columns of the four quadrants of B (cp.async ring, as in the base-product kernel);
//   * a warp reads the four quadrant fragments of each side from shared memory and forms the seven
//     operand fragments in registers (T2 = A21 + A22, T3 = T2 - A11, T4 = A11 - A21, T5 = A12 - T3;
//     S2 = B12 - B11, S3 = B22 - S2, S4 = B22 - B12, S6 = S3 - B21): four adds instead of three more
//     loads per side;
//   * seven FP64 tensor-core accumulator sets (mma.sync m8n8k4), one per product, k ascending;
//   * the epilogue runs the U-chain (U1 = Q0 + Q3, U2 = U1 + Q4, U3 = U1 + Q2; C11 = Q0 + Q1,
//     C12 = U3 + Q5, C21 = U2 - Q6, C22 = U2 + Q2) in registers and stores the four quadrants of C,
//     with the rank-one term of a peeled (odd-size) parent added on the way out.
// The operations on every element are those of the three-launch path (formation, base products,
// recombination); with one warp per tile they also come in the same order and the results have the
// same bits, with two warps per tile each product is the sum of two partial sums over alternate
// 4-deep steps (deterministic, a few ulps from the other order, exact on integer data).
//
// What it costs: every CTA re-reads its row panel of A and column panel of B, so the operands cross
// L2 -> SM about (h / tile) times instead of once, and the seven accumulator sets cap the warp tile
// at 16 x 16 positions.  It pays where the three-launch path is bound by launches and by tiles too
// few to fill the SMs (small n), not where the base products already run near the FP64 peak.
#include "kernels.h"

namespace strassen {

namespace {

template <int WARPS_M_, int WARPS_N_, int KSPLIT_, int MT_, int NT_, int BK_, int STAGES_, int CTAS_, bool DOUBLE_BUFFER_> struct FCfg {
    static constexpr int WARPS_M = WARPS_M_, WARPS_N = WARPS_N_, MT = MT_, NT = NT_, STAGES = STAGES_, CTAS = CTAS_;
    static constexpr int BK = BK_;
    static constexpr bool DOUBLE_BUFFER = DOUBLE_BUFFER_;   // operand fragments of the next 4-deep step fetched before this step's DMMAs
    // KSPLIT warps share one tile of positions and take the 4-deep steps of every slab in turn (their partial
    // products are added through shared memory at the end): two warps per SM sub-partition where the tiles are few.
    static constexpr int KSPLIT = KSPLIT_;
    static constexpr int TILE_WARPS = WARPS_M * WARPS_N;
    static constexpr int TM = WARPS_M * MT * 8, TN = WARPS_N * NT * 8, THREADS = TILE_WARPS * KSPLIT * 32;
    static constexpr int STEPS = BK / 4 / KSPLIT;           // 4-deep steps of a slab per warp
    static constexpr int AS = BK + 4, BS = TN + 4;          // padded rows: conflict-free 8-byte fragment loads
    static constexpr int A_Q = TM * AS, B_Q = BK * BS;      // words of one quadrant's slab
    static constexpr int STAGE_WORDS = 4 * A_Q + 4 * B_Q;
    static constexpr int RED_WORDS = KSPLIT > 1 ? TILE_WARPS * (KSPLIT - 1) * 7 * MT * NT * 2 * 32 : 0;
    static constexpr size_t SMEM_BYTES = size_t(STAGES) * STAGE_WORDS * sizeof(double);
    // loader: a thread copies the 16-byte chunk at one position (row, kc) of A / (krow, nc) of B in A_QPT / B_QPT
    // of the four quadrants, and the same chunk A_ROWS_STEP / B_ROWS_STEP rows further down, A_PASSES / B_PASSES times
    static constexpr int A_POS = TM * (BK / 2), B_POS = BK * (TN / 2);
    static constexpr int A_GROUPS = THREADS >= A_POS ? THREADS / A_POS : 1, A_QPT = 4 / A_GROUPS;
    static constexpr int B_GROUPS = THREADS >= B_POS ? THREADS / B_POS : 1, B_QPT = 4 / B_GROUPS;
    static constexpr int A_PASSES = THREADS >= A_POS ? 1 : A_POS / THREADS, A_ROWS_STEP = THREADS >= A_POS ? TM : THREADS / (BK / 2);
    static constexpr int B_PASSES = THREADS >= B_POS ? 1 : B_POS / THREADS, B_ROWS_STEP = THREADS >= B_POS ? BK : THREADS / (TN / 2);
    static_assert(A_GROUPS * A_QPT == 4 && B_GROUPS * B_QPT == 4 && A_PASSES * A_ROWS_STEP == TM && B_PASSES * B_ROWS_STEP == BK,
                  "the loader covers the slab exactly");
    static_assert(A_GROUPS * A_POS * A_PASSES == (THREADS >= A_POS ? THREADS : A_POS), "every thread has a place in the A loader");
    static_assert(AS % 8 == 4 && BS % 16 == 4 && STAGES >= 2 && STEPS >= 2 && STEPS % 2 == 0, "fragment loads rely on these strides");
    static_assert(RED_WORDS <= STAGES * STAGE_WORDS, "the partial products fit in the ring once it has drained");
};
// Tile 16 x 32 positions: 4 warp tiles of 8 x 16, each shared by two warps that alternate over the 4-deep steps.
// h = 256 gives 128 CTAs of 8 warps: two warps per SM sub-partition, which hide each other's latencies (one alone
// kept the tensor pipe 52 % busy: its own operand sums and shared-memory loads sit between its DMMAs).
using FSplit = FCfg<2, 2, 2, 1, 2, 16, 3, 1, true>;
// The same tile with one warp per warp tile: two CTAs per SM do the hiding once the tiles outnumber the SMs.
using FSmall = FCfg<2, 2, 1, 1, 2, 16, 3, 2, true>;
// 8 warps of 16 x 16 positions: tile 32 x 64, for parents with enough tiles to fill the SMs several times.
using FWide = FCfg<2, 4, 1, 2, 2, 16, 3, 1, false>;

__device__ __forceinline__ void cpa16(uint32_t dst, const void *src, int src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cpa16_full(uint32_t dst, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cpa8(uint32_t dst, const void *src, int src_bytes)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cpa_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N> __device__ __forceinline__ void cpa_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

// D += A.B, one warp-wide 8x8x4 FP64 tensor-core operation.  g = lane / 4, q = lane % 4:
// a = A[g][q], b = B[q][g], d0, d1 = D[g][2q], D[g][2q + 1].
__device__ __forceinline__ void dmma1(double &d0, double &d1, double a, double b)
{
    asm("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};\n"
        : "+d"(d0), "+d"(d1)
        : "d"(a), "d"(b));
}

template <class F>
__global__ void __launch_bounds__(F::THREADS, F::CTAS)
fused_step_kernel(const Node *__restrict__ parents, Bases bases, int h, int item0, int peel)
{
    constexpr int TM = F::TM, TN = F::TN, BK = F::BK, AS = F::AS, BS = F::BS, A_Q = F::A_Q, B_Q = F::B_Q;
    constexpr int MT = F::MT, NT = F::NT, STAGES = F::STAGES, STAGE_WORDS = F::STAGE_WORDS, KSPLIT = F::KSPLIT;
    extern __shared__ __align__(16) double smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tw = warp % F::TILE_WARPS, ks = warp / F::TILE_WARPS;      // warp tile; which of the 4-deep steps are mine
    const int wm = tw / F::WARPS_N, wn = tw % F::WARPS_N;
    const int g = lane >> 2, q = lane & 3;
    const uint32_t smem_base = uint32_t(__cvta_generic_to_shared(smem));

    // Programmatic dependent launch: the launch behind this one in the stream may place its CTAs as soon as
    // every CTA of this grid has got here, and each grid waits for the whole grid before it (and for its memory)
    // before its first global access.  A stream of small products then pays the launch and ramp-up of one
    // product under the tail of the one before.  After any other kind of launch the wait returns at once.
    asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const Node nd = parents[item0 + blockIdx.z];
    const double *A = base_ptr(bases, nd.a.base) + nd.a.off;
    const double *B = base_ptr(bases, nd.b.base) + nd.b.off;
    const long long lda = nd.a.ld, ldb = nd.b.ld;
    const int m0 = blockIdx.y * TM, n0 = blockIdx.x * TN;
    // 16-byte copies need every quadrant row to start on a 16-byte boundary
    const bool a16 = ((reinterpret_cast<uintptr_t>(A) & 15) == 0) && ((lda & 1) == 0) && ((h & 1) == 0);
    const bool b16 = ((reinterpret_cast<uintptr_t>(B) & 15) == 0) && ((ldb & 1) == 0) && ((h & 1) == 0);
    const bool interior = a16 && b16 && m0 + TM <= h && n0 + TN <= h;
    const double *safe = reinterpret_cast<const double *>(parents);     // valid, 16-byte aligned: for copies of 0 bytes
    const int ktiles = (h + BK - 1) / BK;

    // loader coordinates and the element offsets of the four quadrants X11, X12, X21, X22
    const int a_pos = tid % (F::A_GROUPS > 1 ? F::A_POS : F::THREADS), a_q0 = F::A_GROUPS > 1 ? (tid / F::A_POS) * F::A_QPT : 0;
    const int b_pos = tid % (F::B_GROUPS > 1 ? F::B_POS : F::THREADS), b_q0 = F::B_GROUPS > 1 ? (tid / F::B_POS) * F::B_QPT : 0;
    const int a_row = a_pos / (BK / 2), a_kc = a_pos % (BK / 2);
    const int b_krow = b_pos / (TN / 2), b_nc = b_pos % (TN / 2);
    const auto aq = [&](int x) { return (long long)(x >> 1) * h * lda + (x & 1) * h; };
    const auto bq = [&](int x) { return (long long)(x >> 1) * h * ldb + (x & 1) * h; };
    const double *pa = A + (long long)(m0 + a_row) * lda + 2 * a_kc;     // advances by BK per slab
    const double *pb = B + (long long)b_krow * ldb + n0 + 2 * b_nc;      // advances by BK rows per slab
    const uint32_t a_dst0 = smem_base + uint32_t((a_row * AS + 2 * a_kc) * 8);
    const uint32_t b_dst0 = smem_base + uint32_t((4 * A_Q + b_krow * BS + 2 * b_nc) * 8);
    int load_kt = 0;

    auto issue_load = [&]() {
        if (load_kt < ktiles) {
            const uint32_t soff = uint32_t((load_kt % STAGES) * STAGE_WORDS * 8);
            const int k0 = load_kt * BK;
            if (interior && k0 + BK <= h) {
#pragma unroll
                for (int p = 0; p < F::A_PASSES; ++p)
#pragma unroll
                    for (int x = a_q0; x < a_q0 + F::A_QPT; ++x)
                        cpa16_full(a_dst0 + soff + uint32_t((x * A_Q + p * F::A_ROWS_STEP * AS) * 8),
                                   pa + aq(x) + (long long)(p * F::A_ROWS_STEP) * lda);
#pragma unroll
                for (int p = 0; p < F::B_PASSES; ++p)
#pragma unroll
                    for (int x = b_q0; x < b_q0 + F::B_QPT; ++x)
                        cpa16_full(b_dst0 + soff + uint32_t((x * B_Q + p * F::B_ROWS_STEP * BS) * 8),
                                   pb + bq(x) + (long long)(p * F::B_ROWS_STEP) * ldb);
            } else {
                const int kvalid = max(0, min(2, h - (k0 + 2 * a_kc)));
#pragma unroll
                for (int p = 0; p < F::A_PASSES; ++p) {
                    const int nv = (m0 + a_row + p * F::A_ROWS_STEP < h) ? kvalid : 0;
#pragma unroll
                    for (int x = a_q0; x < a_q0 + F::A_QPT; ++x) {
                        const double *s = pa + aq(x) + (long long)(p * F::A_ROWS_STEP) * lda;
                        const uint32_t dst = a_dst0 + soff + uint32_t((x * A_Q + p * F::A_ROWS_STEP * AS) * 8);
                        if (a16) {
                            cpa16(dst, nv ? s : safe, nv * 8);
                        } else {
                            cpa8(dst, nv >= 1 ? s : safe, nv >= 1 ? 8 : 0);
                            cpa8(dst + 8, nv >= 2 ? s + 1 : safe, nv >= 2 ? 8 : 0);
                        }
                    }
                }
                const int cvalid = max(0, min(2, h - (n0 + 2 * b_nc)));
#pragma unroll
                for (int p = 0; p < F::B_PASSES; ++p) {
                    const int nv = (k0 + b_krow + p * F::B_ROWS_STEP < h) ? cvalid : 0;
#pragma unroll
                    for (int x = b_q0; x < b_q0 + F::B_QPT; ++x) {
                        const double *s = pb + bq(x) + (long long)(p * F::B_ROWS_STEP) * ldb;
                        const uint32_t dst = b_dst0 + soff + uint32_t((x * B_Q + p * F::B_ROWS_STEP * BS) * 8);
                        if (b16) {
                            cpa16(dst, nv ? s : safe, nv * 8);
                        } else {
                            cpa8(dst, nv >= 1 ? s : safe, nv >= 1 ? 8 : 0);
                            cpa8(dst + 8, nv >= 2 ? s + 1 : safe, nv >= 2 ? 8 : 0);
                        }
                    }
                }
            }
            pa += BK;
            pb += (long long)BK * ldb;
            ++load_kt;
        }
        cpa_commit();
    };

    double acc[7][MT][NT][2];
#pragma unroll
    for (int j = 0; j < 7; ++j)
#pragma unroll
        for (int i = 0; i < MT; ++i)
#pragma unroll
            for (int t = 0; t < NT; ++t) acc[j][i][t][0] = acc[j][i][t][1] = 0.0;

    // The seven operand fragments of one 4-deep step on each side, formed in registers from the four quadrant fragments.
    const double *a_frag0 = smem + (wm * MT * 8 + g) * AS + q;
    const double *b_frag0 = smem + 4 * A_Q + q * BS + wn * NT * 8 + g;
    auto load_frags = [&](int slot, int kk, double (&ta)[MT][7], double (&sb)[NT][7]) {
        const double *As = a_frag0 + slot * STAGE_WORDS + kk * 4, *Bs = b_frag0 + slot * STAGE_WORDS + kk * 4 * BS;
#pragma unroll
        for (int i = 0; i < MT; ++i) {
            const double *p = As + i * 8 * AS;
            const double a11 = p[0], a12 = p[A_Q], a21 = p[2 * A_Q], a22 = p[3 * A_Q];
            const double t2 = a21 + a22, t3 = t2 - a11;
            ta[i][0] = a11; ta[i][1] = a12; ta[i][2] = t2; ta[i][3] = t3;
            ta[i][4] = a11 - a21; ta[i][5] = a12 - t3; ta[i][6] = a22;
        }
#pragma unroll
        for (int t = 0; t < NT; ++t) {
            const double *p = Bs + t * 8;
            const double b11 = p[0], b12 = p[B_Q], b21 = p[2 * B_Q], b22 = p[3 * B_Q];
            const double s2 = b12 - b11, s3 = b22 - s2;
            sb[t][0] = b11; sb[t][1] = b21; sb[t][2] = s2; sb[t][3] = s3;
            sb[t][4] = b22 - b12; sb[t][5] = b22; sb[t][6] = s3 - b21;
        }
    };
    auto mma_step = [&](const double (&ta)[MT][7], const double (&sb)[NT][7]) {
#pragma unroll
        for (int j = 0; j < 7; ++j)
#pragma unroll
            for (int i = 0; i < MT; ++i)
#pragma unroll
                for (int t = 0; t < NT; ++t) dmma1(acc[j][i][t][0], acc[j][i][t][1], ta[i][j], sb[t][j]);
    };

#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) issue_load();
    cpa_wait<STAGES - 2>();         // slab 0 has landed
    __syncthreads();

    if (F::DOUBLE_BUFFER) {
        // Fragments double-buffered in registers: those of the warp's next step (of the next slab, across the
        // barrier) are fetched and summed before this step's DMMAs are issued.
        double ta0[MT][7], sb0[NT][7], ta1[MT][7], sb1[NT][7];
        int slot = 0;
        load_frags(slot, ks, ta0, sb0);
        for (int kt = 0; kt < ktiles; ++kt) {
#pragma unroll
            for (int i = 0; i < F::STEPS; i += 2) {
                load_frags(slot, ks + KSPLIT * (i + 1), ta1, sb1);
                mma_step(ta0, sb0);
                if (i == 0) issue_load();       // refills the slot every warp left at the last barrier
                if (i + 2 < F::STEPS) {
                    load_frags(slot, ks + KSPLIT * (i + 2), ta0, sb0);
                } else {
                    cpa_wait<STAGES - 2>();     // this thread's copies of the next slab are complete
                    __syncthreads();            // ... and everyone's; all reads of this slab have been issued
                    slot = slot + 1 == STAGES ? 0 : slot + 1;
                    load_frags(slot, ks, ta0, sb0);     // past the last slab: stale data, never used
                }
                mma_step(ta1, sb1);
            }
        }
    } else {
        for (int kt = 0; kt < ktiles; ++kt) {
            if (kt > 0) {
                cpa_wait<STAGES - 2>();
                __syncthreads();
            }
            issue_load();
#pragma unroll
            for (int i = 0; i < F::STEPS; ++i) {
                double ta[MT][7], sb[NT][7];
                load_frags(kt % STAGES, ks + KSPLIT * i, ta, sb);
                mma_step(ta, sb);
            }
        }
    }
    cpa_wait<0>();
    if (KSPLIT > 1) {
        // the warps that took the later steps hand their partial products over through the drained ring
        __syncthreads();
        constexpr int PER_WARP = 7 * MT * NT * 2 * 32;
        if (ks > 0) {
            double *red = smem + ((ks - 1) * F::TILE_WARPS + tw) * PER_WARP + lane;
#pragma unroll
            for (int j = 0; j < 7; ++j)
#pragma unroll
                for (int i = 0; i < MT; ++i)
#pragma unroll
                    for (int t = 0; t < NT; ++t)
#pragma unroll
                        for (int e = 0; e < 2; ++e) red[(((j * MT + i) * NT + t) * 2 + e) * 32] = acc[j][i][t][e];
        }
        __syncthreads();
        if (ks > 0) return;
#pragma unroll
        for (int s2 = 1; s2 < KSPLIT; ++s2) {
            const double *red = smem + ((s2 - 1) * F::TILE_WARPS + tw) * PER_WARP + lane;
#pragma unroll
            for (int j = 0; j < 7; ++j)
#pragma unroll
                for (int i = 0; i < MT; ++i)
#pragma unroll
                    for (int t = 0; t < NT; ++t)
#pragma unroll
                        for (int e = 0; e < 2; ++e) acc[j][i][t][e] += red[(((j * MT + i) * NT + t) * 2 + e) * 32];
        }
    }

    // U-chain in registers, four quadrants of C out
    double *C = base_ptr(bases, nd.c.base) + nd.c.off;
    const long long ldc = nd.c.ld, hq = (long long)h * ldc;
    const bool c16 = ((reinterpret_cast<uintptr_t>(C) & 15) == 0) && ((ldc & 1) == 0) && ((h & 1) == 0);
    const double *acol = A + 2 * h;                              // peeled parent: A[:, 2h] and B[2h, :]
    const double *brow = B + (long long)(2 * h) * ldb;
#pragma unroll
    for (int i = 0; i < MT; ++i) {
        const int r = m0 + (wm * MT + i) * 8 + g;
        if (r >= h) continue;
        double a0 = 0.0, a1 = 0.0;
        if (peel) {
            a0 = acol[(long long)r * lda];
            a1 = acol[(long long)(r + h) * lda];
        }
#pragma unroll
        for (int t = 0; t < NT; ++t) {
            const int c = n0 + (wn * NT + t) * 8 + 2 * q;
            if (c >= h) continue;
            double v[4][2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const double q0 = acc[0][i][t][e], q1 = acc[1][i][t][e], q2 = acc[2][i][t][e], q3 = acc[3][i][t][e];
                const double q4 = acc[4][i][t][e], q5 = acc[5][i][t][e], q6 = acc[6][i][t][e];
                const double u1 = q0 + q3, u2 = u1 + q4, u3 = u1 + q2;
                v[0][e] = q0 + q1;
                v[1][e] = u3 + q5;
                v[2][e] = u2 - q6;
                v[3][e] = u2 + q2;
            }
            const bool two = c + 1 < h;
            if (peel) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    if (e == 1 && !two) break;
                    const double b0 = brow[c + e], b1 = brow[c + e + h];
                    v[0][e] = fma(a0, b0, v[0][e]);
                    v[1][e] = fma(a0, b1, v[1][e]);
                    v[2][e] = fma(a1, b0, v[2][e]);
                    v[3][e] = fma(a1, b1, v[3][e]);
                }
            }
            double *o = C + (long long)r * ldc + c;
            double *dst[4] = {o, o + h, o + hq, o + hq + h};
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                if (two && c16) {
                    *reinterpret_cast<double2 *>(dst[x]) = make_double2(v[x][0], v[x][1]);
                } else {
                    dst[x][0] = v[x][0];
                    if (two) dst[x][1] = v[x][1];
                }
            }
        }
    }
}

template <class F> cudaError_t configure_one()
{
    return cudaFuncSetAttribute(fused_step_kernel<F>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(F::SMEM_BYTES));
}

template <class F>
void launch_one(const Node *parents, const Bases &bases, int h, int64_t item0, int64_t zn, int peel, cudaStream_t stream)
{
    const dim3 grid(unsigned((h + F::TN - 1) / F::TN), unsigned((h + F::TM - 1) / F::TM), unsigned(zn));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(F::THREADS);
    cfg.dynamicSmemBytes = F::SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, fused_step_kernel<F>, parents, bases, h, int(item0), peel);
}

}  // namespace

cudaError_t configure_fused_step_kernels()
{
    cudaError_t e = configure_one<FSplit>();
    if (e == cudaSuccess) e = configure_one<FSmall>();
    if (e == cudaSuccess) e = configure_one<FWide>();
    return e;
}

static bool fused_step_uses_wide_tiles(int64_t h, int64_t count, int sms)
{
    // the wide tile moves half the operand bytes per flop; it needs enough tiles to keep every SM busy
    const int64_t wide_tiles = ((h + FWide::TM - 1) / FWide::TM) * ((h + FWide::TN - 1) / FWide::TN) * count;
    return wide_tiles >= 2 * int64_t(sms);
}

cudaError_t launch_fused_step(const Node *tab, const Launch &op, const Bases &bases, int sm_count, cudaStream_t stream,
                              int *launched)
{
    const Node *parents = tab + op.parent_tab;
    const bool wide = fused_step_uses_wide_tiles(op.h, op.count, sm_count);
    for (int64_t item0 = 0; item0 < op.count; item0 += kMaxItemsPerLaunch) {
        const int64_t zn = op.count - item0 < kMaxItemsPerLaunch ? op.count - item0 : kMaxItemsPerLaunch;
        const int64_t small_tiles = ((op.h + FSmall::TM - 1) / FSmall::TM) * ((op.h + FSmall::TN - 1) / FSmall::TN) * zn;
        if (wide) launch_one<FWide>(parents, bases, int(op.h), item0, zn, op.peel_fused, stream);
        else if (small_tiles <= sm_count) launch_one<FSplit>(parents, bases, int(op.h), item0, zn, op.peel_fused, stream);
        else launch_one<FSmall>(parents, bases, int(op.h), item0, zn, op.peel_fused, stream);
        ++*launched;
    }
    return cudaGetLastError();
}

}  // namespace strassen
