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
cudaError_t launch_form_one(const Node *tab, const Launch &op, const Bases &bases, bool vec, cudaStream_t stream,
                            int *launched);
cudaError_t launch_accumulate(const Node *tab, const Launch &op, const Bases &bases, bool vec, cudaStream_t stream,
                              int *launched);
cudaError_t launch_peel(const Node *tab, const Launch &op, const Bases &bases, cudaStream_t stream, int *launched);
cudaError_t launch_gemm(const Node *tab, const Launch &op, const Bases &bases, int sm_count, cudaStream_t stream,
                        int *launched);

// Kernels one replay of `op` launches (host arithmetic only; mirrors the launchers).
int launches_of(const Launch &op);

cudaError_t probe_fp64(int kind, long long iters, cudaStream_t stream, double *tflops_out);

// Sets the calling thread's error text (what strassen_last_error() returns).
void set_last_error(const char *msg);

}  // namespace strassen
