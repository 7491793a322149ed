// Randomised Hadamard transform kernels (Algorithm 1's RandomHadamardTransform and
// Appendix F's rotation of the activations).
#include "common.cuh"

namespace higgs {

namespace {

// Loads the 32 values of this lane (see fwht1024_warp for the mapping) from a
// row-major source of bf16 or fp32.
template <typename T>
__device__ __forceinline__ void load_group(const T* __restrict__ src, int lane, float (&v)[32]);

template <>
__device__ __forceinline__ void load_group<__nv_bfloat16>(const __nv_bfloat16* __restrict__ src, int lane,
                                                          float (&v)[32]) {
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        uint4 q = __ldg(reinterpret_cast<const uint4*>(src + c * 256 + lane * 8));
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            v[c * 8 + 2 * e] = __uint_as_float(w[e] << 16);
            v[c * 8 + 2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
        }
    }
}

template <>
__device__ __forceinline__ void load_group<float>(const float* __restrict__ src, int lane, float (&v)[32]) {
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        float4 a = __ldg(reinterpret_cast<const float4*>(src + c * 256 + lane * 8));
        float4 b = __ldg(reinterpret_cast<const float4*>(src + c * 256 + lane * 8 + 4));
        v[c * 8 + 0] = a.x; v[c * 8 + 1] = a.y; v[c * 8 + 2] = a.z; v[c * 8 + 3] = a.w;
        v[c * 8 + 4] = b.x; v[c * 8 + 5] = b.y; v[c * 8 + 6] = b.z; v[c * 8 + 7] = b.w;
    }
}

// One warp per (token, group): x+ = (H/32) diag(sign) x, written as fp16 in "fragment order": inside every block of
// 64 inputs the 32 input pairs are permuted so that the eight pairs one lane of the product kernel needs as
// m16n8k16 B-fragment registers (steps m = 0..3, halves h = 0..1 of its column pair t) are 32 contiguous bytes:
// position t*8 + m*2 + h holds pair 8m + t + 4h.  Extra threads beyond the transform work clear `zero_ptr` (the fp32
// accumulation target of a K-split product) so no separate memset launch is needed.
template <typename T>
__global__ void __launch_bounds__(256) rht_activations_kernel(const T* __restrict__ x, __half* __restrict__ xdag,
                                                              int64_t B, int64_t K, uint64_t xi,
                                                              float* __restrict__ zero_ptr, size_t zero_floats) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t groups = K / kGroup;
    const size_t gtid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t gthreads = (size_t)gridDim.x * blockDim.x;
    pdl_trigger();     // the product kernel may start its table build and weight prefetch now
    pdl_wait();        // x may be the previous kernel's output; the buffers written below may still be read by it
    for (size_t i = gtid; i < zero_floats; i += gthreads) zero_ptr[i] = 0.0f;
    if (warp >= B * groups) return;
    const int64_t b = warp / groups, gi = warp % groups;
    float v[32];
    load_group<T>(x + b * K + gi * kGroup, lane, v);
    apply_signs1024(v, xi, gi * kGroup, lane);
    fwht1024_warp(v, lane);
    uint32_t* dst = reinterpret_cast<uint32_t*>(xdag + b * K + gi * kGroup);
    // this lane's chunk c holds inputs c*256 + lane*8 .. +7: pairs 4j + i (i = 0..3) of 64-input block c*4 + lane/8,
    // j = lane % 8, i.e. m = j >> 1, h = j & 1, t = i  ->  position i*8 + j
    const int j = lane & 7;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        uint32_t* blk = dst + (c * 4 + (lane >> 3)) * 32;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            __half2 h = __floats2half2_rn(v[c * 8 + 2 * e] * 0.03125f, v[c * 8 + 2 * e + 1] * 0.03125f);
            blk[e * 8 + j] = *reinterpret_cast<uint32_t*>(&h);
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(256) rht_debug_kernel(const T* __restrict__ x, float* __restrict__ out,
                                                        int64_t rows, int64_t K, uint64_t xi, float mul) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t groups = K / kGroup;
    if (warp >= rows * groups) return;
    const int64_t b = warp / groups, gi = warp % groups;
    float v[32];
    load_group<T>(x + b * K + gi * kGroup, lane, v);
    apply_signs1024(v, xi, gi * kGroup, lane);
    fwht1024_warp(v, lane);
    float* dst = out + b * K + gi * kGroup;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        *reinterpret_cast<float4*>(dst + c * 256 + lane * 8) =
            make_float4(v[c * 8] * mul, v[c * 8 + 1] * mul, v[c * 8 + 2] * mul, v[c * 8 + 3] * mul);
        *reinterpret_cast<float4*>(dst + c * 256 + lane * 8 + 4) =
            make_float4(v[c * 8 + 4] * mul, v[c * 8 + 5] * mul, v[c * 8 + 6] * mul, v[c * 8 + 7] * mul);
    }
}

}  // namespace

int launch_rht_activations(const higgs_desc& d, const void* x, int64_t B, __half* xdag, float* zero_ptr,
                           size_t zero_floats, cudaStream_t st) {
    const int64_t warps = B * (d.K / kGroup);
    int64_t blocks = (warps + 7) / 8;
    if (zero_floats) {
        int64_t zb = (int64_t)((zero_floats + 256 * 8 - 1) / (256 * 8));
        if (zb > 1184) zb = 1184;
        if (zb > blocks) blocks = zb;
    }
    return cuda_status(launch_pdl(rht_activations_kernel<__nv_bfloat16>, dim3((unsigned)blocks), dim3(256), 0, st,
                                  static_cast<const __nv_bfloat16*>(x), xdag, B, d.K, d.rht_seed, zero_ptr, zero_floats));
}

int launch_rht_debug(const higgs_desc& d, const void* x, int x_dtype, int64_t rows, float* out, int normalised,
                     cudaStream_t st) {
    const int64_t warps = rows * (d.K / kGroup);
    if (warps == 0) return HIGGS_OK;
    const unsigned blocks = (unsigned)((warps + 7) / 8);
    const float mul = normalised ? 0.03125f : 1.0f;
    if (x_dtype == HIGGS_BF16)
        rht_debug_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(x), out, rows, d.K,
                                                               d.rht_seed, mul);
    else if (x_dtype == HIGGS_F32)
        rht_debug_kernel<float><<<blocks, 256, 0, st>>>(static_cast<const float*>(x), out, rows, d.K, d.rht_seed, mul);
    else
        return HIGGS_ERR_UNSUPPORTED;
    return cuda_status(cudaGetLastError());
}

}  // namespace higgs
