// Small device utilities behind the C ABI: the launch-latency floor, seeded Gaussian samples for the grid fit.
#include "common.cuh"

namespace higgs {

namespace {

// Does nothing, launched like the product kernels (programmatic dependent launch, same block shape and dynamic
// shared memory): the time of a chain of these is what a chain of product launches costs before any byte moves.
__global__ void floor_kernel() {
    pdl_trigger();
    pdl_wait();
}

// Sample i, coordinate k of N(0, I_p): Box-Muller on two 24-bit uniforms cut from output number i p + k of the
// splitmix64 stream seeded with `seed` (the generator the sign function uses).
__global__ void gaussian_samples_kernel(int p, uint64_t seed, int64_t count, float* __restrict__ out) {
    const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= count) return;
    const uint64_t z = sign_word(seed, (uint64_t)c);
    const float u1 = ((float)(uint32_t)(z >> 40) + 0.5f) * (1.0f / 16777216.0f);
    const float u2 = ((float)(uint32_t)((z >> 16) & 0xffffffu) + 0.5f) * (1.0f / 16777216.0f);
    out[c] = sqrtf(-2.0f * logf(u1)) * cospif(2.0f * u2);
}

// Ordinary (fully stream-ordered) empty kernel: see launch_stream_fence.
__global__ void fence_kernel() {}

}  // namespace

// Ends a producer of packed codes, scales or grids.  A product kernel enqueued next may start early, but then it
// overlaps only this empty kernel, which itself started after the producer's kernels had completed and their
// writes were visible: the product's early reads of its weights are ordered after the producer's writes.
int launch_stream_fence(cudaStream_t st) {
    fence_kernel<<<1, 32, 0, st>>>();
    return cuda_status(cudaGetLastError());
}

int launch_floor(int blocks, int threads, size_t smem, cudaStream_t st) {
    static int configured[64] = {0};
    const int ok = device_once(configured, [] {
        return cudaFuncSetAttribute(floor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448) == cudaSuccess ? 1 : -1;
    });
    if (ok < 0) return HIGGS_ERR_CUDA;
    return cuda_status(launch_pdl(floor_kernel, dim3((unsigned)blocks), dim3((unsigned)threads), smem, st));
}

int launch_gaussian_samples(int p, uint64_t seed, int64_t m, float* out, cudaStream_t st) {
    const int64_t count = m * p;
    gaussian_samples_kernel<<<(unsigned)((count + 255) / 256), 256, 0, st>>>(p, seed, count, out);
    return cuda_status(cudaGetLastError());
}

}  // namespace higgs
