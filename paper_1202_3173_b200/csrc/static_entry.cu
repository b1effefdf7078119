// strassen_dgemm_static: one Strassen-Winograd level for callers that cannot allocate device
// memory.  Its temporaries (the eight operand sums, the seven products and the node table the
// kernels index) live in a file-scope device array instead of a cudaMalloc'd workspace.
#include "strassen_b200.h"

#include <atomic>
#include <string>

#include "kernels.h"
#include "plan.h"

using namespace strassen;

namespace {

constexpr int64_t kMaxN = STRASSEN_STATIC_MAX_N;
constexpr int64_t kMaxH = kMaxN / 2;
constexpr int64_t kTableWords = 64;                         // 8 nodes of 48 bytes (384 of the 512 bytes reserved)
constexpr int64_t kMatWords = kMaxH * kMaxH;                // one quarter-size matrix at the largest n
constexpr int64_t kScratchWords = kTableWords + 15 * kMatWords;

// Held by every device that loads the library, until the process exits (about 7.9 MB).
// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) double g_static_scratch[kScratchWords];

constexpr int kMaxDevices = 64;
// Device address of g_static_scratch and SM count, per device ordinal.  Atomics: two host threads may make
// their first call on a device at once; both then resolve the same values, and the pointer is published last.
std::atomic<double *> g_scratch_ptr[kMaxDevices];
std::atomic<int> g_sm_count[kMaxDevices];

// Writes the node table of a one-level tree: entry 0 is the parent (A, B, C as given), entries
// 1..7 its children j = 0..6 (Appendix A): quadrant operands point into A / B, operand sums
// and products into the scratch array.
__global__ void static_nodes_kernel(Node *tab, int n, int h, int ldw, long long mat, long long ws0)
{
    const int t = threadIdx.x;
    if (t > 7) return;
    Node nd;
    if (t == 0) {
        nd.a = Operand{0, n, BASE_A};
        nd.b = Operand{0, n, BASE_B};
        nd.c = Operand{0, n, BASE_C};
    } else {
        const int j = t - 1;
        // A-side: T0 = A11, T1 = A12, T6 = A22 are views; T2..T5 are sums in slots 0..3
        const long long a12 = h, a22 = (long long)h * n + h;
        if (j == 0) nd.a = Operand{0, n, BASE_A};
        else if (j == 1) nd.a = Operand{a12, n, BASE_A};
        else if (j == 6) nd.a = Operand{a22, n, BASE_A};
        else nd.a = Operand{ws0 + (j - 2) * mat, ldw, BASE_WS};
        // B-side: S0 = B11, S1 = B21, S5 = B22 are views; S2, S3, S4, S6 are sums in slots 4..7
        const long long b21 = (long long)h * n, b22 = (long long)h * n + h;
        if (j == 0) nd.b = Operand{0, n, BASE_B};
        else if (j == 1) nd.b = Operand{b21, n, BASE_B};
        else if (j == 5) nd.b = Operand{b22, n, BASE_B};
        else nd.b = Operand{ws0 + (4 + (j == 6 ? 3 : j - 2)) * mat, ldw, BASE_WS};
        nd.c = Operand{ws0 + (8 + j) * mat, ldw, BASE_WS};
    }
    tab[t] = nd;
}

int static_fail(int status, const std::string &msg)
{
    set_last_error(msg.c_str());     // read back through strassen_last_error()
    return status;
}

}  // namespace

extern "C" int strassen_dgemm_static(int64_t n, const double *A, const double *B, double *C, void *stream_v)
{
    set_last_error("");
    if (!A || !B || !C) return static_fail(STRASSEN_INVALID_ARG, "A, B and C must be non-NULL");
    if (n < 2) return static_fail(STRASSEN_INVALID_ARG, "n must be at least 2 (one recursion level is always taken)");
    if (n > kMaxN) {
        return static_fail(STRASSEN_WORKSPACE_TOO_SMALL,
                           "n = " + std::to_string(n) + " exceeds STRASSEN_STATIC_MAX_N = " + std::to_string(kMaxN) +
                               ": the static scratch array holds the temporaries of at most that size");
    }
    const uintptr_t bits = reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(B) | reinterpret_cast<uintptr_t>(C);
    if (bits & 7) return static_fail(STRASSEN_MISALIGNED, "A, B and C must be 8-byte aligned");
    const uintptr_t bytes = uintptr_t(n) * uintptr_t(n) * 8;
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(A), b0 = reinterpret_cast<uintptr_t>(B), c0 = reinterpret_cast<uintptr_t>(C);
    if ((c0 < a0 + bytes && a0 < c0 + bytes) || (c0 < b0 + bytes && b0 < c0 + bytes))
        return static_fail(STRASSEN_ALIAS, "C overlaps A or B");

    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return static_fail(STRASSEN_CUDA_ERROR, std::string("cudaGetDevice: ") + cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices) return static_fail(STRASSEN_INVALID_ARG, "device ordinal out of range");
    if (!g_scratch_ptr[dev].load(std::memory_order_acquire)) {
        // First call on this device: resolve the device address of the scratch array (with this
        // device current), read the SM count, opt the product kernels in to their shared memory.
        // None of these allocates.
        double *ptr = nullptr;
        e = cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_static_scratch);
        if (e != cudaSuccess || !ptr)
            return static_fail(STRASSEN_CUDA_ERROR, std::string("cudaGetSymbolAddress(static scratch): ") + cudaGetErrorString(e));
        int sms = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return static_fail(STRASSEN_CUDA_ERROR, std::string("cudaDeviceGetAttribute: ") + cudaGetErrorString(e));
        e = configure_gemm_kernels();        // shared-memory attribute of the product kernels: no allocation either
        if (e != cudaSuccess) return static_fail(STRASSEN_CUDA_ERROR, std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e));
        g_sm_count[dev].store(sms, std::memory_order_relaxed);
        g_scratch_ptr[dev].store(ptr, std::memory_order_release);
    }
    double *scratch = g_scratch_ptr[dev].load(std::memory_order_acquire);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);

    const int64_t h = n / 2;
    const int64_t ldw = (h + 3) / 4 * 4;
    const int64_t mat = (h * ldw + 31) / 32 * 32;           // at most kMatWords for h <= 256
    if (kTableWords + 15 * mat > kScratchWords) return static_fail(STRASSEN_WORKSPACE_TOO_SMALL, "temporaries exceed the static scratch array");

    Node *tab = reinterpret_cast<Node *>(scratch);
    static_nodes_kernel<<<1, 8, 0, stream>>>(tab, int(n), int(h), int(ldw), (long long)mat, (long long)kTableWords);
    e = cudaGetLastError();
    if (e != cudaSuccess) return static_fail(STRASSEN_CUDA_ERROR, std::string("node table kernel: ") + cudaGetErrorString(e));

    Bases bases;
    bases.p[BASE_A] = const_cast<double *>(A);
    bases.p[BASE_B] = const_cast<double *>(B);
    bases.p[BASE_C] = C;
    bases.p[BASE_WS] = scratch;
    const bool vec = ((bits & 15) == 0) && (n % 2 == 0) && (h % 2 == 0);

    Launch form{};
    form.kind = OP_FORM; form.level = 0; form.j = -1; form.vec_ok = vec;
    form.parent_tab = 0; form.child_tab = 1; form.count = 1; form.m = n; form.h = h;
    Launch gemm{};
    gemm.kind = OP_GEMM; gemm.level = 1; gemm.j = -1; gemm.vec_ok = 1;
    gemm.parent_tab = 1; gemm.child_tab = -1; gemm.count = 7; gemm.m = h; gemm.h = 0;
    Launch rec = form;
    rec.kind = OP_RECOMBINE;
    Launch peel = form;
    peel.kind = OP_PEEL; peel.vec_ok = 0;

    int launched = 0;
    e = launch_form(tab, form, bases, vec, stream, &launched);
    if (e == cudaSuccess) e = launch_gemm(tab, gemm, bases, g_sm_count[dev].load(std::memory_order_relaxed), stream, &launched);
    if (e == cudaSuccess) e = launch_recombine(tab, rec, bases, vec, stream, &launched);
    if (e == cudaSuccess && (n & 1)) e = launch_peel(tab, peel, bases, stream, &launched);
    if (e != cudaSuccess) return static_fail(STRASSEN_CUDA_ERROR, std::string("kernel launch: ") + cudaGetErrorString(e));
    return STRASSEN_OK;
}
