// pop_prefill_scores_noalloc: the prefill importance scores (Eq. 3) for callers that must not
// allocate device memory.  The two temporaries of the scoring pipeline (down-projection column
// norms and per-channel activation energies, 2 x N doubles) live in a fixed file-scope device
// array instead of stream-ordered allocations; the kernels are the library's ordinary ones.
#include <mutex>

#include "pop_common.cuh"

// Scratch shared by every call on a device: [0, MAX_N) column norms, [MAX_N, 2 MAX_N) energies.
// 512 KB per GPU that loads the library, held until the process exits.
static __device__ __align__(256) double g_noalloc_scratch[2 * POP_NOALLOC_MAX_N];

// In host code `g_noalloc_scratch` is only a handle for the runtime, not a device address: the
// address of the array on each device is looked up once, with that device current.
static constexpr int MAX_DEVICES = 64;
static double* g_scratch_addr[MAX_DEVICES];
static std::mutex g_scratch_mutex;

static int scratch_for_current_device(double** out) {
    int dev = -1;
    POP_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEVICES) return POP_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        double* p = nullptr;
        POP_CUDA(cudaGetSymbolAddress((void**)&p, g_noalloc_scratch));
        if (!p) return POP_ERR_CUDA;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return POP_OK;
}

extern "C" int pop_prefill_scores_noalloc(const void* X, int L, int d, const void* Wg, const void* Wu,
                                          const void* Wd, int N, pop_dtype_t dtype, double* scores_out,
                                          void* cuda_stream) {
    if (!X || !Wg || !Wu || !Wd || !scores_out || L <= 0 || d <= 0 || N <= 0) return POP_ERR_INVALID_ARG;
    if (dtype != POP_F32 && dtype != POP_BF16) return POP_ERR_UNSUPPORTED;
    if (N > POP_NOALLOC_MAX_N) {
        pop_set_cuda_error(cudaErrorInvalidValue,
                           "pop_prefill_scores_noalloc: N is larger than POP_NOALLOC_MAX_N, the size of the fixed scratch array");
        return POP_ERR_UNSUPPORTED;
    }
    const size_t row = (size_t)d * (dtype == POP_F32 ? 4 : 2);
    if (row % 16 != 0 || row > 65536) return POP_ERR_UNSUPPORTED;
    const uintptr_t bits = (uintptr_t)X | (uintptr_t)Wg | (uintptr_t)Wu | (uintptr_t)Wd;
    if ((bits & 15u) != 0 || ((uintptr_t)scores_out & 7u) != 0) return POP_ERR_INVALID_ARG;

    double* scratch = nullptr;
    int rc = scratch_for_current_device(&scratch);
    if (rc != POP_OK) return rc;
    double* norm = scratch;                        // every entry below N is overwritten: nothing to clear
    double* s2 = scratch + POP_NOALLOC_MAX_N;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    rc = pop_launch_colnorm(Wd, d, N, dtype, norm, st);
    if (rc == POP_OK) rc = pop_launch_prefill_s2_exact(X, L, d, Wg, Wu, N, dtype, nullptr, N, s2, st);
    if (rc == POP_OK) rc = pop_launch_scores(s2, norm, N, scores_out, nullptr, st);
    return rc;
}
