// hbfp_gemm_static: the BFP GEMM for callers that must not allocate device memory.
//
// hbfp_gemm needs a caller-provided workspace (packed copies of the operands, split-K partial
// tiles). Some callers cannot provide one: a plug-in running inside a host framework that has
// already claimed all device memory for its own pool, a serving loop in which any allocation is
// forbidden because it would synchronise the device, code that runs while another component
// holds the allocator. For them this entry point keeps the workspace inside the library, in a
// fixed array in device memory that exists from the moment the library is loaded on a GPU until
// the process exits. Nothing is allocated or freed by the call.
#include "common.cuh"

#include <atomic>

namespace {

// The built-in workspace. Every GPU that loads the library carries these bytes until exit.
static __device__ __align__(256) unsigned char g_static_workspace[HBFP_STATIC_WORKSPACE_BYTES];

// Device address of the array, per device. In host code the array's name only stands for the
// symbol; the address a kernel can use has to be asked for, with that device current.
// Host threads may make their first calls at the same time: the cache is atomic (they would all
// store the same address).
constexpr int kMaxDevices = 64;
std::atomic<void*> g_workspace_ptr[kMaxDevices];

int static_workspace(void** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return HBFP_ERR_CUDA;
    void* p = g_workspace_ptr[dev].load(std::memory_order_acquire);
    if (!p) {
        if (cudaGetSymbolAddress(&p, g_static_workspace) != cudaSuccess || !p) return HBFP_ERR_CUDA;
        g_workspace_ptr[dev].store(p, std::memory_order_release);
    }
    *out = p;
    return HBFP_OK;
}

}  // namespace

extern "C" int hbfp_gemm_static(int transA, int transB, int64_t M, int64_t N, int64_t K, const float* A,
                                int64_t lda, const float* B, int64_t ldb, float* C, int64_t ldc,
                                const hbfp_format* fmtA, const hbfp_format* fmtB, uint32_t flags, void* stream) {
    size_t need = 0;
    int rc = hbfp_gemm_workspace(transA, transB, M, N, K, fmtA, fmtB, &need);
    if (rc) return rc;
    if (need > (size_t)HBFP_STATIC_WORKSPACE_BYTES) return HBFP_ERR_STATIC_LIMIT;
    void* ws = nullptr;
    rc = static_workspace(&ws);
    if (rc) return rc;
    // Nothing in the workspace has to start at zero: the quantisers overwrite every byte the GEMM
    // reads (they clear the padding they document as zero themselves) and split-K partial tiles
    // are fully written before they are summed.
    return hbfp_gemm(transA, transB, M, N, K, A, lda, B, ldb, C, ldc, fmtA, fmtB, ws,
                     (size_t)HBFP_STATIC_WORKSPACE_BYTES, flags, stream);
}
