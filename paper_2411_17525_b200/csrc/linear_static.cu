// higgs_linear for callers that cannot hand the library a workspace.
//
// Some callers cannot allocate device memory: code that runs in a real-time loop or another
// context where cudaMalloc is forbidden, plugins that only receive input and output
// tensors from their host framework, and processes whose memory pool is owned by someone
// else.  For them the scratch that higgs_linear needs (the rotated activations and, for some
// shapes, an fp32 staging copy of the output) lives in one fixed array inside the library
// image.  Every GPU that loads the library carries that array until the process exits, which
// is why it is kept small and why requests that do not fit are refused.
#include "common.cuh"

#include <mutex>

namespace higgs {
namespace {

constexpr size_t kStaticScratchBytes = 4u << 20;   // 4 MiB: every Llama-shaped layer up to 28672 x 8192 at B <= 16

// Host code must never use this name as a pointer: on the host it is only a handle for
// cudaGetSymbolAddress.  Device code may name it directly.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_setup_mutex;
void* g_scratch_ptr[64] = {nullptr};   // device address of the array, per device ordinal

// Looks the array's device address up once per device (the calling thread's current device).
int static_scratch(void** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return HIGGS_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return HIGGS_ERR_CUDA;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return HIGGS_OK;
}

}  // namespace
}  // namespace higgs

extern "C" {

size_t higgs_linear_static_capacity(void) { return higgs::kStaticScratchBytes; }

int higgs_linear_static(const higgs_desc* desc, const void* x, int64_t B, const void* packed, const void* scales,
                        const float* grid, void* y, int y_dtype, void* stream) {
    const int rc = higgs::check_desc(desc);
    if (rc != HIGGS_OK) return rc;
    if (B < 0) return HIGGS_ERR_INVALID_ARG;
    if (B == 0 || desc->N == 0) return HIGGS_OK;
    const size_t need = higgs_workspace_bytes(desc, HIGGS_OP_LINEAR, B);
    if (need == 0) return HIGGS_ERR_UNSUPPORTED;
    if (need > higgs::kStaticScratchBytes) return HIGGS_ERR_STATIC_SCRATCH;   // refused before anything is enqueued
    void* scratch = nullptr;
    const int sc = higgs::static_scratch(&scratch);
    if (sc != HIGGS_OK) return sc;
    // The kernels overwrite every scratch byte they later read (rotated activations) and clear the
    // accumulation target themselves, so stale contents of an earlier call are harmless.
    return higgs_linear(desc, x, B, packed, scales, grid, y, y_dtype, scratch, higgs::kStaticScratchBytes, stream);
}

}  // extern "C"
