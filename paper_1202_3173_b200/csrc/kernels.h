// Internal launch interface between the C ABI (api.cu) and the kernels.
#pragma once
#include <cuda_runtime.h>

#include "plan.h"

namespace strassen {

// The four allocations node operands refer to: A, B (never written), C, workspace.
struct Bases {
    double *p[4];
};

// Select chain instead of a dynamic index: keeps the kernel argument out of local memory.
__host__ __device__ __forceinline__ double *base_ptr(const Bases &b, int id)
{
    return id == BASE_A ? b.p[0] : id == BASE_B ? b.p[1] : id == BASE_C ? b.p[2] : b.p[3];
}

// Every launcher enqueues on `stream`, adds the number of kernels it launched to
// *launched, and returns the status of the last launch.
cudaError_t launch_form(const Node *tab, const Launch &op, const Bases &bases, bool vec, cudaStream_t stream,
                        int *launched);
cudaError_t launch_recombine(const Node *tab, const Launch &op, const Bases &bases, bool vec, cudaStream_t stream,
                             int *launched);
cudaError_t launch_form2(const Node *tab, const Launch &op, const Bases &bases, bool vec, cudaStream_t stream, int *launched);
cudaError_t launch_recombine2(const Node *tab, const Launch &op, const Bases &bases, bool vec, cudaStream_t stream,
                              int *launched);
// Two BFS levels in one pass where the children have odd size.
cudaError_t launch_form2_odd(const Node *tab, const Launch &op, const Bases &bases, cudaStream_t stream, int *launched);
cudaError_t launch_recombine2_odd(const Node *tab, const Launch &op, const Bases &bases, cudaStream_t stream, int *launched);
// Items (gridDim.z) one launch of a streaming kernel covers; longer lists are cut into several launches.
constexpr int kMaxItemsPerLaunch = 32768;

// Three BFS levels in one pass (add3_kernels.cu).
cudaError_t launch_form3(const Node *tab, const Launch &op, const Bases &bases, cudaStream_t stream, int *launched);
cudaError_t launch_recombine3(const Node *tab, const Launch &op, const Bases &bases, cudaStream_t stream, int *launched);
cudaError_t launch_form_one(const Node *tab, const Launch &op, const Bases &bases, bool vec, cudaStream_t stream,
                            int *launched);
cudaError_t launch_accumulate(const Node *tab, const Launch &op, const Bases &bases, bool vec, cudaStream_t stream,
                              int *launched);
cudaError_t launch_peel(const Node *tab, const Launch &op, const Bases &bases, cudaStream_t stream, int *launched);
cudaError_t launch_gemm(const Node *tab, const Launch &op, const Bases &bases, int sm_count, cudaStream_t stream,
                        int *launched);

// Thin products over `count` nodes (full inner dimension K): columns [c0, c0 + nc) for rows [0, rows),
// and rows [r0, r0 + nr) for columns [0, cols); nc, nr <= 8.
cudaError_t launch_thin_cols(const Node *nodes, const Bases &bases, int K, int rows, int c0, int nc, int64_t count,
                             cudaStream_t stream, int *launched);
cudaError_t launch_thin_rows(const Node *nodes, const Bases &bases, int K, int cols, int r0, int nr, int64_t count,
                             cudaStream_t stream, int *launched);
// The same for the seven children (size h, leaves[7 p + j]) of each of `count` BFS parents, from the parents' quadrants:
// columns [M, M + rem) for all rows and rows [M, M + rem) for columns [0, M) of every child's product.
cudaError_t launch_thin_siblings(const Node *parents, const Node *leaves, const Bases &bases, int h, int M, int rem, int64_t count,
                                 cudaStream_t stream, int *launched);

// A base product whose size is 1..8 past a multiple of 64 is computed as a tiled bulk of that
// multiple plus thin products for the remainder rows / columns; returns the remainder (0 = none).
inline int gemm_thin_remainder(int64_t m)
{
    const int rem = int(m % 64);
    return rem >= 1 && rem <= 8 ? rem : 0;
}

// The thin remainders of base products that are whole sets of siblings are computed per parent (from its quadrants).
inline bool gemm_thin_siblings(const Launch &op)
{
    return op.sibling_tab > 0 && op.count % 7 == 0 && gemm_thin_remainder(op.m) != 0 && op.m > 64;
}

// How the tiled part of a batch of `count` base products with output extent M is launched on a device
// with `sms` SMs: all leaves on the 64 x 64 tiling (two CTAs per SM), or `wide_leaves` leaves on the
// 128 x 128 tiling followed by the rest on the 64 x 64 tiling.
struct GemmSplit {
    bool all_small;
    int64_t wide_leaves;
};
inline GemmSplit gemm_split(int64_t M, int64_t count, int sms)
{
    // Few large tiles leave SMs idle: when the 128 x 128 tiling cannot give every SM a tile, the 64 x 64
    // tiling is compared by rounds x tile cost (a 128 x 128 tile alone on an SM = 8 units).
    const int64_t tpl_wide = ((M + 127) / 128) * ((M + 127) / 128), tpl_small = ((M + 63) / 64) * ((M + 63) / 64);
    const int64_t t_wide = tpl_wide * count, t_small = tpl_small * count;
    const int64_t cost_wide = ((t_wide + sms - 1) / sms) * 8;
    const int64_t cost_small = t_small <= sms ? 2 : ((t_small + 2 * sms - 1) / (2 * sms)) * 4 + 1;
    if (cost_small * 10 < cost_wide * 9) return GemmSplit{true, 0};
    // The last, partly filled round of 128 x 128 tiles costs a whole tile time.  When it is less than half
    // full, the leaves it belongs to go to the 64 x 64 tiling instead: full rounds of large tiles first, then
    // a short launch of quarter-size tiles spread over all SMs.
    const int64_t full_rounds = t_wide / sms, left = t_wide - full_rounds * sms;
    int64_t wide_leaves = count;
    if (full_rounds >= 4 && left > 0 && 2 * left < sms) {
        wide_leaves = full_rounds * sms / tpl_wide;
        if ((count - wide_leaves) * tpl_small > 2 * int64_t(sms)) wide_leaves = count;   // tail too long to pay off
    }
    return GemmSplit{false, wide_leaves};
}

// One tiled launch of the base products: the block [row0, row_end) x [col0, col_end) of C for the leaves
// [first, first + leaves), on the 128 x 128 tiling or the 64 x 64 one.
struct GemmRegion {
    bool small;
    int row0, col0, row_end, col_end;
    int64_t first, leaves;
};
// The tiled launches that cover the M x M output of `count` leaves.  Where M ends 1..64 past a multiple of
// 128, the 128 x 128 tiling would spend whole tiles on that margin; the leaves on that tiling then take the
// margin as a right and a bottom strip of 64 x 64 tiles (worth it from a few full rounds of strip tiles on).
// Writes at most 4 entries to `out` and returns their number.
inline int gemm_regions(int64_t M64, int64_t count, int sms, GemmRegion *out)
{
    const int M = int(M64);
    int k = 0;
    const int margin = M % 128, bulk = M - margin;
    bool strips = false;
    if (margin >= 1 && margin <= 64 && bulk > 0) {
        // rounds x tile cost in eighteenths of a 128 x 128 tile time: such a tile alone on an SM costs 18, a
        // 64 x 64 tile beside another one 10 (two per SM, a little slower per flop), a launch's ramp 2
        const auto rounds = [](int64_t tiles, int64_t slots) { return (tiles + slots - 1) / slots; };
        const int64_t tw = (M + 127) / 128, ts = (M + 63) / 64, tb = bulk / 128, strip_tiles = 2 * (bulk / 64) + 1;
        const int64_t whole_wide = rounds(tw * tw * count, sms) * 18;
        const int64_t whole_small = rounds(ts * ts * count, 2 * sms) * 10 + 2;
        const int64_t with_strips = rounds(tb * tb * count, sms) * 18 + rounds(strip_tiles * count, 2 * sms) * 10 + 4;
        strips = strip_tiles * count >= 4 * int64_t(sms) && with_strips < whole_wide && with_strips < whole_small;
    }
    if (!strips && gemm_split(M, count, sms).all_small) {
        out[k++] = GemmRegion{true, 0, 0, M, M, 0, count};
        return k;
    }
    const int wide_extent = strips ? bulk : M;
    const GemmSplit split = gemm_split(wide_extent, count, sms);       // which leaves fill whole rounds of large tiles
    const int64_t wide_leaves = split.all_small ? count : split.wide_leaves;
    out[k++] = GemmRegion{false, 0, 0, wide_extent, wide_extent, 0, wide_leaves};
    if (strips) {
        out[k++] = GemmRegion{true, 0, bulk, bulk, M, 0, wide_leaves};     // right strip
        out[k++] = GemmRegion{true, bulk, 0, M, M, 0, wide_leaves};        // bottom strip with the corner
    }
    if (wide_leaves < count) out[k++] = GemmRegion{true, 0, 0, M, M, wide_leaves, count - wide_leaves};
    return k;
}
// One whole BFS step in one kernel (fused_step.cu): op.count parents of size 2 op.h (+ 1 when peeled).
cudaError_t launch_fused_step(const Node *tab, const Launch &op, const Bases &bases, int sm_count, cudaStream_t stream,
                              int *launched);
cudaError_t configure_fused_step_kernels();
// The fused step replaces three launches whose base products cannot fill the SMs with large tiles: it pays while
// the children's 128 x 128 tiles number fewer than the SMs (measured on B200).
inline bool fused_step_pays(int64_t h, int64_t parents, int sms)
{
    const int64_t tiles = ((h + 127) / 128) * ((h + 127) / 128) * 7 * parents;
    return tiles < sms;
}

// Generic bilinear schemes (bilinear.cu): one linear-combination launch over op.count parents.
struct LinComb;
cudaError_t launch_lincomb(const Node *tab, const Launch &op, const LinComb &lc, const Bases &bases, bool vec, cudaStream_t stream,
                           int *launched);

// A launch on 64 x 64 tiles that cannot fill the two CTA slots of every SM runs on 32 x 64 tiles instead.
inline bool gemm_uses_tiny_tiles(int64_t tiles64, int sms) { return tiles64 < 2 * int64_t(sms); }

constexpr int kNominalSMs = 148;   // B200; used where launches are counted without a device at hand

// Sets the shared-memory attribute of every GEMM kernel shape on the current device (idempotent).
cudaError_t configure_gemm_kernels();

// Diagonal scaling passes around the product (scale_kernels.cu).
cudaError_t launch_scale_in(const PlanDesc &d, const Bases &bases, cudaStream_t stream, int *launched);
cudaError_t launch_scale_out(const PlanDesc &d, const Bases &bases, cudaStream_t stream, int *launched);
int scale_launches(const PlanDesc &d, bool in);

// Kernels one replay of `op` launches (host arithmetic only; mirrors the launchers).
int launches_of(const Launch &op);

cudaError_t probe_fp64(int kind, long long iters, cudaStream_t stream, double *tflops_out);

// Sets the calling thread's error text (what strassen_last_error() returns).
void set_last_error(const char *msg);

}  // namespace strassen
