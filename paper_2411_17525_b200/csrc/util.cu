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

// Sums `world` fp32 slots of `count` values in slot order (a fixed order: the result is reproducible) into y.
__global__ void reduce_slots_kernel(const float* __restrict__ slots, int world, int64_t count, void* __restrict__ y, int bf16) {
    pdl_trigger();
    pdl_wait();
    const int64_t quads = count / 4;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < quads; i += (int64_t)gridDim.x * blockDim.x) {
        float4 acc = *reinterpret_cast<const float4*>(slots + 4 * i);
        for (int r = 1; r < world; ++r) {
            const float4 v = *reinterpret_cast<const float4*>(slots + (int64_t)r * count + 4 * i);
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        if (bf16) {
            const __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
            reinterpret_cast<uint2*>(y)[i] = make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
        } else {
            reinterpret_cast<float4*>(y)[i] = acc;
        }
    }
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

int launch_reduce_slots(const float* slots, int world, int64_t count, void* y, int y_dtype, cudaStream_t st) {
    int64_t blocks = (count / 4 + 255) / 256;
    if (blocks > 1184) blocks = 1184;
    if (blocks < 1) blocks = 1;
    return cuda_status(launch_pdl(reduce_slots_kernel, dim3((unsigned)blocks), dim3(256), 0, st, slots, world, count, y,
                                  y_dtype == HIGGS_BF16 ? 1 : 0));
}

// t^2 = ||W^ - W||^2 / ||W||^2 from the two accumulated sums (0 for an all-zero layer)
__global__ void error_ratio_kernel(double* sums) { sums[2] = sums[1] > 0.0 ? sums[0] / sums[1] : 0.0; }

int launch_error_ratio(double* sums, cudaStream_t st) {
    error_ratio_kernel<<<1, 1, 0, st>>>(sums);
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
