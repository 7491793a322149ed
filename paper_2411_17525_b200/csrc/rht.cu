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

// Four warps per (token, group), one block of 128 threads each: x+ = (H/32) diag(sign) x, written as fp16 in "fragment
// order": inside every block of 64 inputs the 32 input pairs are permuted so that the eight pairs one lane of the
// product kernel needs as m16n8k16 B-fragment registers (steps m = 0..3, halves h = 0..1 of its column pair t) are 32
// contiguous bytes: position t*8 + m*2 + h holds pair 8m + t + 4h.  Warp q of the block owns inputs 256 q .. + 255 of
// the group, 8 per lane: butterflies over those 8 in registers, over the 32 lanes by shuffles, over the 4 warps
// through shared memory (the transform is on the latency path between two dependent product launches, so it is
// spread over four warps instead of one).  Threads also clear `zero_ptr` (the fp32 accumulation target of a K-split
// product) so that no separate memset launch is needed.
template <typename T>
__global__ void __launch_bounds__(128) rht_activations_kernel(const T* __restrict__ x, __half* __restrict__ xdag,
                                                              int64_t B, int64_t K, uint64_t xi,
                                                              float* __restrict__ zero_ptr, size_t zero_floats) {
    __shared__ __align__(16) float ex[4][256];
    const int lane = threadIdx.x & 31, q = threadIdx.x >> 5;
    const int64_t groups = K / kGroup;
    const size_t gtid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t gthreads = (size_t)gridDim.x * blockDim.x;
    pdl_trigger();     // the product kernel may start its table build and weight prefetch now
    pdl_wait();        // x may be the previous kernel's output; the buffers written below may still be read by it
    for (size_t i = gtid; i < zero_floats; i += gthreads) zero_ptr[i] = 0.0f;
    if ((int64_t)blockIdx.x >= B * groups) return;           // (blocks beyond the transform work only clear)
    const int64_t b = blockIdx.x / groups, gi = blockIdx.x % groups;
    const int64_t k0 = gi * kGroup + q * 256 + lane * 8;     // this lane's 8 consecutive inputs
    float v[8];
    {
        const T* src = x + b * K + k0;
        if (sizeof(T) == 2) {
            const uint4 q4 = __ldg(reinterpret_cast<const uint4*>(src));
            const uint32_t w4[4] = {q4.x, q4.y, q4.z, q4.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                v[2 * e] = __uint_as_float(w4[e] << 16);
                v[2 * e + 1] = __uint_as_float(w4[e] & 0xffff0000u);
            }
        } else {
            const float4 a = __ldg(reinterpret_cast<const float4*>(src)), c = __ldg(reinterpret_cast<const float4*>(src) + 1);
            v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = c.x; v[5] = c.y; v[6] = c.z; v[7] = c.w;
        }
        const uint32_t bits = (uint32_t)(sign_word(xi, (uint64_t)k0 >> 6) >> ((uint64_t)k0 & 63ull)) & 0xffu;
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = __uint_as_float(__float_as_uint(v[e]) ^ (((bits >> e) & 1u) << 31));
    }
#pragma unroll
    for (int h = 1; h < 8; h <<= 1) {
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            if ((r & h) == 0) { const float a = v[r], c = v[r | h]; v[r] = a + c; v[r | h] = a - c; }
        }
    }
#pragma unroll
    for (int m = 1; m < 32; m <<= 1) {
        const bool upper = (lane & m) != 0;
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            const float o = __shfl_xor_sync(0xffffffffu, v[r], m);
            v[r] = upper ? (o - v[r]) : (v[r] + o);
        }
    }
    *reinterpret_cast<float4*>(&ex[q][lane * 8]) = make_float4(v[0], v[1], v[2], v[3]);
    *reinterpret_cast<float4*>(&ex[q][lane * 8 + 4]) = make_float4(v[4], v[5], v[6], v[7]);
    __syncthreads();
    float o[8];
#pragma unroll
    for (int r = 0; r < 8; ++r) o[r] = 0.f;
#pragma unroll
    for (int qq = 0; qq < 4; ++qq) {
        const float4 u0 = *reinterpret_cast<const float4*>(&ex[qq][lane * 8]);
        const float4 u1 = *reinterpret_cast<const float4*>(&ex[qq][lane * 8 + 4]);
        const float sgn = (__popc(q & qq) & 1) ? -1.f : 1.f;
        o[0] = fmaf(sgn, u0.x, o[0]); o[1] = fmaf(sgn, u0.y, o[1]); o[2] = fmaf(sgn, u0.z, o[2]); o[3] = fmaf(sgn, u0.w, o[3]);
        o[4] = fmaf(sgn, u1.x, o[4]); o[5] = fmaf(sgn, u1.y, o[5]); o[6] = fmaf(sgn, u1.z, o[6]); o[7] = fmaf(sgn, u1.w, o[7]);
    }
    // this lane holds pairs 4 j + i (i = 0..3, j = lane % 8) of 64-input block q*4 + lane/8 of the group, i.e.
    // m = j >> 1, h = j & 1, t = i  ->  position i*8 + j
    uint32_t* blk = reinterpret_cast<uint32_t*>(xdag + b * K + gi * kGroup) + (q * 4 + (lane >> 3)) * 32;
    const int j = lane & 7;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const __half2 hh = __floats2half2_rn(o[2 * e] * 0.03125f, o[2 * e + 1] * 0.03125f);
        blk[e * 8 + j] = *reinterpret_cast<const uint32_t*>(&hh);
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
    int64_t blocks = B * (d.K / kGroup);                   // one block of four warps per (token, group)
    if (zero_floats) {
        int64_t zb = (int64_t)((zero_floats + 128 * 8 - 1) / (128 * 8));
        if (zb > 1184) zb = 1184;
        if (zb > blocks) blocks = zb;
    }
    return cuda_status(launch_pdl(rht_activations_kernel<__nv_bfloat16>, dim3((unsigned)blocks), dim3(128), 0, st,
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
