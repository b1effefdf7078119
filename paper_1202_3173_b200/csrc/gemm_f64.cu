// Batched FP64 base-case products Q = T.S for all live leaves in one launch
// (Algorithm 2 "localStrassen" at its cutoff; Section 5.4: classical multiply below n0).
//
// sm_100a has no FP64 kind in tcgen05.mma, so the tensor-core route for this contraction is
// the warp-level DMMA, mma.sync m8n8k4 with FP64 accumulators in registers (the larger f64
// shapes issue the same number of native 8x8x4 operations and run at the same rate).  Design:
//   * persistent CTAs (one per SM, 256 threads = 8 warps as 2 x 4), static round-robin over
//     the flattened list of 128 x 128 output tiles of all leaves; tiles of one leaf are
//     adjacent so that CTAs running together share its operand panels through L2;
//   * operands staged by cp.async into a 4-stage shared-memory ring of 128x16 (A) and
//     16x128 (B) slabs; the ring runs continuously across tiles, so the loads of the next
//     tile are in flight while the current one finishes;
//   * one barrier per 16-deep slab, placed before the last quarter of the slab's DMMAs, and
//     the first fragments of the next slab are read right after it, so that no warp waits
//     for shared-memory latency with an empty tensor pipe;
//   * rows padded (+4 doubles) so that the 8-byte fragment loads of a half-warp fall in 16
//     distinct bank pairs;
//   * each warp owns 64 x 32 of the tile: 8 x 4 DMMA accumulators of 8 x 8;
//   * the last slab of a tile is computed strip by strip of 8 rows, and every finished strip is
//     stored while the next one is computed, so the tile's stores drain beside tensor work;
//   * interior slabs of 16-byte-aligned operands take a branch-free copy path; ragged edges
//     (size not a multiple of 128 / 16) are zero-filled by cp.async's src-size operand and
//     masked in the epilogue; operands that are only 8-byte aligned (views into matrices
//     with an odd leading dimension) use 8-byte copies.
#include "kernels.h"

#include <atomic>

namespace strassen {

namespace {

// Tile shape variants: BM x BN CTA tile, each warp owns WTM x 32 of it (warps are BM/WTM x BN/32),
// BK-deep slabs, STAGES slabs in the ring, CTAS resident per SM.
template <int BM_, int BN_, int WTM_, int BK_, int STAGES_, int CTAS_> struct Cfg {
    static constexpr int BM = BM_, BN = BN_, WTM = WTM_, BK = BK_, STAGES = STAGES_, CTAS = CTAS_;
    static constexpr int WARPS_N = BN / 32, THREADS = (BM / WTM) * WARPS_N * 32;
    static constexpr int MT = WTM / 8;                // DMMA accumulator tiles along m per warp
    static constexpr int AS = BK + 4;                 // padded row of the A slab (doubles)
    static constexpr int BS = BN + 4;                 // padded row of the B slab
    static constexpr int A_STAGE = BM * AS, B_STAGE = BK * BS;
    static constexpr int STAGE_WORDS = A_STAGE + B_STAGE;
    static constexpr size_t SMEM_BYTES = size_t(STAGES) * STAGE_WORDS * sizeof(double);
    static constexpr int A_KCHUNKS = BK / 2;                    // 16-byte chunks per A row
    static constexpr int A_ROWS_STEP = THREADS / A_KCHUNKS;     // rows covered by one pass of all threads
    static constexpr int A_CHUNKS = BM / A_ROWS_STEP;           // passes (chunks per thread) for the A slab
    static constexpr int B_KROWS_STEP = THREADS / (BN / 2);     // B rows covered by one pass
    static constexpr int B_CHUNKS = BK / B_KROWS_STEP;          // passes for the B slab
    static_assert(BK % 8 == 0 && (AS % 16 == 4 || AS % 16 == 12) && BS % 16 == 4, "fragment loads rely on these strides");
};
// Measured alternatives that did not beat CfgWide on 343 x 512^3 (33.9 TFLOP/s): 128 x 64 tiles with two
// CTAs per SM (32.7), 32-deep slabs (33.9), 8-deep slabs (32.7), 64 x 128 tiles with 16 warps per SM (33.9).
// Storing the whole tile after its last slab cost 2.4 us per tile (of 71 us at K = 512); interleaved with the
// last slab as below, and with the tile position stepped instead of divided out, 1.1 us remain.  Also measured
// without gain: half the tile staged in shared memory for bulk-copy stores; mbarriers in place of the per-slab
// CTA barrier (warps free to drift: per-tile cost down, steady state 1 % slower).
using CfgWide = Cfg<128, 128, 64, 16, 4, 1>;    // 8 warps of 64 x 32; 149.5 KB of shared memory, one CTA per SM
using CfgSmall = Cfg<64, 64, 32, 16, 4, 2>;     // 4 warps of 32 x 32; 54 KB: four times as many tiles, for launches
                                                // whose 128 x 128 tiles would leave most SMs idle
using CfgTiny = Cfg<32, 64, 16, 16, 4, 3>;      // 4 warps of 16 x 32; 40 KB: eight times as many tiles, for launches whose
                                                // 64 x 64 tiles would not even fill the two CTA slots of every SM

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, int src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async16_full(uint32_t dst, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async8(uint32_t dst, const void *src, int src_bytes)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

// D += A.B, one warp-wide 8x8x4 FP64 tensor-core operation.  g = lane / 4, q = lane % 4:
// a = A[g][q], b = B[q][g], d0, d1 = D[g][2q], D[g][2q + 1].
__device__ __forceinline__ void dmma(double &d0, double &d1, double a, double b)
{
    asm("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};\n"
        : "+d"(d0), "+d"(d1)
        : "d"(a), "d"(b));
}

struct TileCoord {
    int node, m0, n0;
};

// Position of a CTA in the flattened tile list: leaf and tile within the leaf.  A CTA visits tiles
// blockIdx.x, blockIdx.x + gridDim.x, ...; stepping (node, r) by the quotient and remainder of
// gridDim.x / tiles_per_node keeps the 64-bit division out of the loop.
struct TileWalk {
    int node, r;
};

// Per-thread source state of the tile currently being loaded; a and b advance slab by slab.
struct LoadState {
    const double *a;        // element (m0 + row0, k0 + 2 kc) of A: this thread's first chunk of the slab
    const double *b;        // element (k0 + krow0, n0 + 2 nc) of B
    long long a_step;       // A_ROWS_STEP rows of A
    long long b_step;       // B_KROWS_STEP rows of B
    int a_rows_ok;          // bit i: row m0 + row0 + A_ROWS_STEP i lies inside the block
    int b_cols;             // valid columns of this thread's B chunk: 0, 1 or 2
    bool a16, b16;          // 16-byte copies legal
    bool interior;          // all rows / columns valid and both operands 16-byte aligned
};

// LAST_STEPS: the 4-deep steps of a tile's last 16-deep slab that hold data.  Where K leaves 1..8 columns in
// it (771 = 48 x 16 + 3: one step) the steps that would multiply zero fill are not issued.  (Taking the short
// slab first instead, so that the stores still drain beside four steps, measured no gain at all.)
template <class C, int LAST_STEPS = C::BK / 4>
__global__ void __launch_bounds__(C::THREADS, C::CTAS)
gemm_f64_kernel(const Node *__restrict__ nodes, Bases bases, GemmRegion reg, int K, int tiles_n, int tiles_per_node, int ktiles,
                long long total_tiles)
{
    // reg: the block of every leaf's output computed here (tiles are counted from its corner); K: inner dimension.
    constexpr int BM = C::BM, BN = C::BN, WTM = C::WTM, MT = C::MT, BK = C::BK, AS = C::AS, BS = C::BS, STAGES = C::STAGES, STAGE_WORDS = C::STAGE_WORDS;
    constexpr int A_STAGE = C::A_STAGE, A_CHUNKS = C::A_CHUNKS, A_ROWS_STEP = C::A_ROWS_STEP, A_KCHUNKS = C::A_KCHUNKS;
    constexpr int B_CHUNKS = C::B_CHUNKS, B_KROWS_STEP = C::B_KROWS_STEP;
    extern __shared__ __align__(16) double smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int wm = warp / C::WARPS_N, wn = warp % C::WARPS_N;   // 2 x WARPS_N warps
    const int g = lane >> 2, q = lane & 3;            // DMMA fragment coordinates
    const uint32_t smem_base = uint32_t(__cvta_generic_to_shared(smem));

    // loader coordinates: A chunk (row, kc) = (tid / A_KCHUNKS + A_ROWS_STEP i, tid % A_KCHUNKS);
    // B chunk (krow, nc) = (tid / (BN / 2) + B_KROWS_STEP i, tid % (BN / 2))
    const int a_row0 = tid / A_KCHUNKS, a_kc = tid % A_KCHUNKS;
    const int b_krow0 = tid / (BN / 2), b_nc = tid % (BN / 2);
    const uint32_t a_dst0 = smem_base + uint32_t((a_row0 * AS + a_kc * 2) * 8);
    const uint32_t b_dst0 = smem_base + uint32_t((A_STAGE + b_krow0 * BS + b_nc * 2) * 8);
    const bool k_ragged = (K % BK) != 0;

    const int my_tiles = int((total_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x);   // the grid never exceeds total_tiles
    const int step_node = int(gridDim.x) / tiles_per_node, step_r = int(gridDim.x) % tiles_per_node;
    auto advance = [&](TileWalk &w) {
        w.node += step_node;
        w.r += step_r;
        if (w.r >= tiles_per_node) {
            w.r -= tiles_per_node;
            ++w.node;
        }
    };
    auto coord = [&](const TileWalk &w) {
        TileCoord c;
        c.node = w.node;
        c.m0 = reg.row0 + (w.r / tiles_n) * BM;
        c.n0 = reg.col0 + (w.r % tiles_n) * BN;
        return c;
    };
    TileWalk load_at{int(blockIdx.x) / tiles_per_node, int(blockIdx.x) % tiles_per_node};
    TileWalk tile_at = load_at;
    int load_left = my_tiles;          // tiles whose loads have not been issued completely
    int load_k = 0;
    LoadState ls;
    const double *safe = reinterpret_cast<const double *>(nodes);   // valid, 16-byte aligned: for copies of 0 bytes

    // The node of the tile whose loads start next is fetched one slab ahead of its use, so that
    // the table read never sits between a warp and its next DMMAs.
    TileCoord next_tc = coord(load_at);
    Operand next_a = nodes[next_tc.node].a, next_b = nodes[next_tc.node].b;

    auto setup_load = [&]() {
        const TileCoord tc = next_tc;
        Node nd;
        nd.a = next_a;
        nd.b = next_b;
        const double *A = base_ptr(bases, nd.a.base) + nd.a.off;
        const double *B = base_ptr(bases, nd.b.base) + nd.b.off;
        ls.a_step = (long long)A_ROWS_STEP * nd.a.ld;
        ls.b_step = (long long)B_KROWS_STEP * nd.b.ld;
        ls.a16 = ((reinterpret_cast<uintptr_t>(A) & 15) == 0) && ((nd.a.ld & 1) == 0);
        ls.b16 = ((reinterpret_cast<uintptr_t>(B) & 15) == 0) && ((nd.b.ld & 1) == 0);
        ls.a_rows_ok = 0;
#pragma unroll
        for (int i = 0; i < A_CHUNKS; ++i)
            if (tc.m0 + a_row0 + A_ROWS_STEP * i < reg.row_end) ls.a_rows_ok |= 1 << i;
        ls.a = A + (long long)(tc.m0 + a_row0) * nd.a.ld + a_kc * 2;
        const int col = tc.n0 + b_nc * 2;
        ls.b_cols = max(0, min(2, reg.col_end - col));
        ls.b = B + (long long)b_krow0 * nd.b.ld + col;
        ls.interior = ls.a16 && ls.b16 && tc.m0 + BM <= reg.row_end && tc.n0 + BN <= reg.col_end;
    };

    auto issue_load = [&](int slot) {
        if (load_left > 0) {
            if (load_k == 0) setup_load();
            const uint32_t soff = uint32_t(slot * STAGE_WORDS * 8);
            if (ls.interior && !(k_ragged && load_k == ktiles - 1)) {
#pragma unroll
                for (int i = 0; i < A_CHUNKS; ++i)
                    cp_async16_full(a_dst0 + soff + uint32_t(A_ROWS_STEP * i * AS * 8), ls.a + i * ls.a_step);
#pragma unroll
                for (int i = 0; i < B_CHUNKS; ++i)
                    cp_async16_full(b_dst0 + soff + uint32_t(B_KROWS_STEP * i * BS * 8), ls.b + i * ls.b_step);
            } else {
                const int k0 = load_k * BK;
                // A slab: BM rows x BK k
                const int kvalid = max(0, min(2, K - (k0 + a_kc * 2)));
#pragma unroll
                for (int i = 0; i < A_CHUNKS; ++i) {
                    const int nv = ((ls.a_rows_ok >> i) & 1) ? kvalid : 0;
                    const double *s = nv ? ls.a + i * ls.a_step : safe;
                    const uint32_t dst = a_dst0 + soff + uint32_t(A_ROWS_STEP * i * AS * 8);
                    if (ls.a16) {
                        cp_async16(dst, s, nv * 8);
                    } else {
                        cp_async8(dst, s, nv >= 1 ? 8 : 0);
                        cp_async8(dst + 8, nv >= 2 ? s + 1 : safe, nv >= 2 ? 8 : 0);
                    }
                }
                // B slab: 16 k x 128 columns
#pragma unroll
                for (int i = 0; i < B_CHUNKS; ++i) {
                    const int nv = (k0 + b_krow0 + B_KROWS_STEP * i) < K ? ls.b_cols : 0;
                    const double *s = nv ? ls.b + i * ls.b_step : safe;
                    const uint32_t dst = b_dst0 + soff + uint32_t(B_KROWS_STEP * i * BS * 8);
                    if (ls.b16) {
                        cp_async16(dst, s, nv * 8);
                    } else {
                        cp_async8(dst, s, nv >= 1 ? 8 : 0);
                        cp_async8(dst + 8, nv >= 2 ? s + 1 : safe, nv >= 2 ? 8 : 0);
                    }
                }
            }
            ls.a += BK;
            ls.b += B_CHUNKS * ls.b_step;
            if (++load_k == ktiles) {
                load_k = 0;
                advance(load_at);
                if (--load_left > 0) {
                    next_tc = coord(load_at);
                    next_a = nodes[next_tc.node].a;
                    next_b = nodes[next_tc.node].b;
                }
            }
        }
        cp_async_commit();
    };

    double acc[MT][4][2];
#pragma unroll
    for (int i = 0; i < MT; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j][0] = acc[i][j][1] = 0.0;

    // fragments of one 4-deep step: A[64 rows of the warp][4 k] and B[4 k][32 columns of the warp]
    const double *a_frag0 = smem + (wm * WTM + g) * AS + q;
    const double *b_frag0 = smem + A_STAGE + q * BS + wn * 32 + g;
    auto load_frags = [&](int slot, int kk, double (&fa)[MT], double (&fb)[4]) {
        const double *As = a_frag0 + slot * STAGE_WORDS + kk * 4;
        const double *Bs = b_frag0 + slot * STAGE_WORDS + kk * 4 * BS;
#pragma unroll
        for (int i = 0; i < MT; ++i) fa[i] = As[i * 8 * AS];
#pragma unroll
        for (int j = 0; j < 4; ++j) fb[j] = Bs[j * 8];
    };
    auto mma_step = [&](const double (&fa)[MT], const double (&fb)[4]) {
#pragma unroll
        for (int i = 0; i < MT; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) dmma(acc[i][j][0], acc[i][j][1], fa[i], fb[j]);
    };

#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) issue_load(s);
    cp_async_wait<STAGES - 2>();      // slab 0 has landed
    __syncthreads();

    double fa0[MT], fb0[4], fa1[MT], fb1[4];
    int slot = 0;
    load_frags(slot, 0, fa0, fb0);

    // One 16-deep slab, 4-deep step by step over all accumulators.
    auto slab_steps = [&]() {
        // Invariant: every warp has passed the barrier of the previous slab, i.e. has finished
        // reading it, so its slot may be refilled; fa0 / fb0 hold step 0 of this slab.
#pragma unroll
        for (int kk = 0; kk < BK / 4; kk += 2) {
            load_frags(slot, kk + 1, fa1, fb1);
            mma_step(fa0, fb0);
            if (kk == 0) issue_load((slot + STAGES - 1) % STAGES);
            if (kk + 2 < BK / 4) {
                load_frags(slot, kk + 2, fa0, fb0);
            } else {
                cp_async_wait<STAGES - 2>();      // this thread's copies of the next slab are complete
                __syncthreads();                  // ... and everyone's; all reads of this slab are done
                slot = slot + 1 == STAGES ? 0 : slot + 1;
                load_frags(slot, 0, fa0, fb0);
            }
            mma_step(fa1, fb1);
        }
    };

    for (int t = 0; t < my_tiles; ++t, advance(tile_at)) {
        const TileCoord tc = coord(tile_at);
        const Operand c_op = nodes[tc.node].c;        // consumed in the last slab
        for (int kt = 0; kt < ktiles - 1; ++kt) slab_steps();

        // The last slab of the tile runs row by row of the warp's accumulators instead (all four
        // steps of one 8-row strip, then the next strip), and each strip is stored while the next
        // one is being computed: the tile's 128 KB of stores drain beside the DMMAs of this slab
        // instead of holding every warp after it.
        double *C = base_ptr(bases, c_op.base) + c_op.off;
        const long long ldc = c_op.ld;
        const bool c16 = ((reinterpret_cast<uintptr_t>(C) & 15) == 0) && ((c_op.ld & 1) == 0);
        const int r0 = tc.m0 + wm * WTM + g, c0 = tc.n0 + wn * 32 + q * 2;
        double *o = C + (long long)r0 * ldc + c0;
        const bool interior_out = c16 && tc.m0 + BM <= reg.row_end && tc.n0 + BN <= reg.col_end;
        auto store_strip = [&](int i) {
            double *e = o + (long long)(i * 8) * ldc;
            if (interior_out) {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    *reinterpret_cast<double2 *>(e + j * 8) = make_double2(acc[i][j][0], acc[i][j][1]);
            } else {
                const int r = r0 + i * 8;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int c = c0 + j * 8;
                    if (r < reg.row_end && c < reg.col_end) {
                        if (c + 1 < reg.col_end) {
                            if (c16) *reinterpret_cast<double2 *>(e + j * 8) = make_double2(acc[i][j][0], acc[i][j][1]);
                            else { e[j * 8] = acc[i][j][0]; e[j * 8 + 1] = acc[i][j][1]; }
                        } else {
                            e[j * 8] = acc[i][j][0];
                        }
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j][0] = acc[i][j][1] = 0.0;
        };
        {
            double fbL[LAST_STEPS][4], faL[2][LAST_STEPS];
            const double *As = a_frag0 + slot * STAGE_WORDS, *Bs = b_frag0 + slot * STAGE_WORDS;
#pragma unroll
            for (int kk = 0; kk < LAST_STEPS; ++kk) {
#pragma unroll
                for (int j = 0; j < 4; ++j) fbL[kk][j] = Bs[kk * 4 * BS + j * 8];
                faL[0][kk] = As[kk * 4];
            }
#pragma unroll
            for (int i = 0; i < MT; ++i) {
                if (i + 1 < MT) {
#pragma unroll
                    for (int kk = 0; kk < LAST_STEPS; ++kk) faL[(i + 1) & 1][kk] = As[(i + 1) * 8 * AS + kk * 4];
                } else {
                    cp_async_wait<STAGES - 2>();      // as in slab_steps: the next slab has landed,
                    __syncthreads();                  // and every read of this one has been issued
                    slot = slot + 1 == STAGES ? 0 : slot + 1;
                }
#pragma unroll
                for (int kk = 0; kk < LAST_STEPS; ++kk)
#pragma unroll
                    for (int j = 0; j < 4; ++j) dmma(acc[i][j][0], acc[i][j][1], faL[i & 1][kk], fbL[kk][j]);
                if (i == 0) issue_load((slot + STAGES - 1) % STAGES);
                if (i >= 1) store_strip(i - 1);
            }
        }
        load_frags(slot, 0, fa0, fb0);
        store_strip(MT - 1);
    }
    cp_async_wait<0>();
}

}  // namespace

namespace {

// Per device: kernels opted in to > 48 KB of dynamic shared memory.  Atomic because two host threads may make
// their first call at once; the set-up itself is idempotent, so both may run it.
std::atomic<bool> g_configured[64];

}  // namespace

cudaError_t configure_gemm_kernels();

namespace {

template <class C, bool SHORT_OK = false>
cudaError_t launch_cfg(const Node *nodes, const Bases &bases, const GemmRegion &reg, int K, int sm_count, cudaStream_t stream)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !g_configured[dev].load(std::memory_order_acquire)) {
        e = configure_gemm_kernels();
        if (e != cudaSuccess) return e;
    }
    const int tiles_m = (reg.row_end - reg.row0 + C::BM - 1) / C::BM, tiles_n = (reg.col_end - reg.col0 + C::BN - 1) / C::BN;
    const int tiles_per_node = tiles_m * tiles_n;
    const int ktiles = (K + C::BK - 1) / C::BK;
    const long long total = (long long)tiles_per_node * reg.leaves;
    const long long slots = (long long)sm_count * C::CTAS;
    const int grid = int(total < slots ? total : slots);
    const int last_steps = (K - (ktiles - 1) * C::BK + 3) / 4;      // 4-deep steps of the last slab that hold data
    const Node *first = nodes + reg.first;
    if (SHORT_OK && last_steps == 1)
        gemm_f64_kernel<C, SHORT_OK ? 1 : C::BK / 4><<<grid, C::THREADS, C::SMEM_BYTES, stream>>>(first, bases, reg, K, tiles_n, tiles_per_node, ktiles, total);
    else if (SHORT_OK && last_steps == 2)
        gemm_f64_kernel<C, SHORT_OK ? 2 : C::BK / 4><<<grid, C::THREADS, C::SMEM_BYTES, stream>>>(first, bases, reg, K, tiles_n, tiles_per_node, ktiles, total);
    else
        gemm_f64_kernel<C><<<grid, C::THREADS, C::SMEM_BYTES, stream>>>(first, bases, reg, K, tiles_n, tiles_per_node, ktiles, total);
    return cudaGetLastError();
}

}  // namespace

cudaError_t configure_gemm_kernels()
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && g_configured[dev].load(std::memory_order_acquire)) return cudaSuccess;
    e = cudaFuncSetAttribute(gemm_f64_kernel<CfgWide>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(CfgWide::SMEM_BYTES));
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(gemm_f64_kernel<CfgWide, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(CfgWide::SMEM_BYTES));
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(gemm_f64_kernel<CfgWide, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(CfgWide::SMEM_BYTES));
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(gemm_f64_kernel<CfgSmall>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(CfgSmall::SMEM_BYTES));
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(gemm_f64_kernel<CfgTiny>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(CfgTiny::SMEM_BYTES));
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) g_configured[dev].store(true, std::memory_order_release);
    return cudaSuccess;
}

cudaError_t launch_gemm(const Node *tab, const Launch &op, const Bases &bases, int sm_count, cudaStream_t stream,
                        int *launched)
{
    // A size a few elements past a multiple of 64 would spend a whole extra row and column of tiles on
    // those elements: the tiles cover the multiple, thin products the remainder.
    const int K = int(op.m), rem = gemm_thin_remainder(op.m), M = K - rem;
    const Node *nodes = tab + op.parent_tab;
    cudaError_t err = cudaSuccess;
    if (M > 0) {
        GemmRegion regions[4];
        const int nreg = gemm_regions(M, op.count, sm_count, regions);
        for (int i = 0; i < nreg && err == cudaSuccess; ++i) {
            ++*launched;
            const GemmRegion &r = regions[i];
            const int64_t tiles64 = int64_t((r.row_end - r.row0 + 63) / 64) * ((r.col_end - r.col0 + 63) / 64) * r.leaves;
            if (!r.small) err = launch_cfg<CfgWide, true>(nodes, bases, r, K, sm_count, stream);
            else if (gemm_uses_tiny_tiles(tiles64, sm_count)) err = launch_cfg<CfgTiny>(nodes, bases, r, K, sm_count, stream);
            else err = launch_cfg<CfgSmall>(nodes, bases, r, K, sm_count, stream);
        }
        if (err != cudaSuccess) return err;
    }
    if (rem && gemm_thin_siblings(op))
        return launch_thin_siblings(tab + (op.sibling_tab - 1), nodes, bases, K, M, rem, op.count / 7, stream, launched);
    if (rem) {
        err = launch_thin_cols(nodes, bases, K, K, M, rem, op.count, stream, launched);     // columns [M, K), all rows
        if (err != cudaSuccess) return err;
        if (M > 0) err = launch_thin_rows(nodes, bases, K, M, M, rem, op.count, stream, launched);   // rows [M, K), columns [0, M)
    }
    return err;
}

}  // namespace strassen
