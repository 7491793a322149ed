// Dequantisation to the original space (Appendix F, "Dequantization"): for every (row, group)
//   r = scale * G[codes]  (the layer in the rotated space),   w^ = diag(sign) (H / sqrt(g)) r.
// Validation / export path, not on the decode hot path (which never leaves the rotated space).
#include "common.cuh"

namespace higgs {

namespace {

// The dequantised group (row, gi) in registers: lane l gets the 32 elements idx = c*256 + l*8 + e of the group (the
// mapping of fwht1024_warp), so its codes are 4 runs of 8/p consecutive canonical codes.
template <int P>
__device__ __forceinline__ void dequantize_group(const uint8_t* __restrict__ canonical, const __half* __restrict__ scales,
                                                 const float* __restrict__ grid, int64_t K, uint64_t xi, int64_t row, int64_t gi,
                                                 int lane, float (&v)[32]) {
    const int64_t groups = K / kGroup;
    const float scale = __half2float(scales[((row / kRowTile) * groups + gi) * kRowTile + (row % kRowTile)]);   // tile-major
    const uint8_t* crow = canonical + row * (K / P) + gi * (kGroup / P);
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const int e0 = c * 256 + lane * 8;                 // first element of the chunk inside the group
        if (P == 2) {
            const uint32_t w = *reinterpret_cast<const uint32_t*>(crow + e0 / 2);      // 4 codes = 8 elements
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const float2 gp = __ldg(reinterpret_cast<const float2*>(grid) + ((w >> (8 * t)) & 0xffu));
                v[c * 8 + 2 * t] = scale * gp.x;
                v[c * 8 + 2 * t + 1] = scale * gp.y;
            }
        } else {
            const uint2 w = *reinterpret_cast<const uint2*>(crow + e0);               // 8 codes = 8 elements
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                const uint32_t code = ((t < 4 ? w.x : w.y) >> (8 * (t & 3))) & 0xffu;
                v[c * 8 + t] = scale * __ldg(grid + code);
            }
        }
    }
    fwht1024_warp(v, lane);
#pragma unroll
    for (int r = 0; r < 32; ++r) v[r] *= 0.03125f;          // H / sqrt(1024)
    apply_signs1024(v, xi, gi * kGroup, lane);
}

// One warp per (row, group of 1024).
template <int P, typename OutT>
__global__ void __launch_bounds__(256) dequantize_kernel(const uint8_t* __restrict__ canonical, const __half* __restrict__ scales,
                                                         const float* __restrict__ grid, OutT* __restrict__ W_out,
                                                         int64_t N, int64_t K, uint64_t xi) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t groups = K / kGroup;
    if (warp >= N * groups) return;
    const int64_t row = warp / groups, gi = warp % groups;
    float v[32];
    dequantize_group<P>(canonical, scales, grid, K, xi, row, gi, lane, v);
    OutT* dst = W_out + row * K + gi * kGroup;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        if (sizeof(OutT) == 4) {
            float* d = reinterpret_cast<float*>(dst) + c * 256 + lane * 8;
            *reinterpret_cast<float4*>(d) = make_float4(v[c * 8], v[c * 8 + 1], v[c * 8 + 2], v[c * 8 + 3]);
            *reinterpret_cast<float4*>(d + 4) = make_float4(v[c * 8 + 4], v[c * 8 + 5], v[c * 8 + 6], v[c * 8 + 7]);
        } else {
            uint32_t w4[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                __nv_bfloat162 h = __floats2bfloat162_rn(v[c * 8 + 2 * e], v[c * 8 + 2 * e + 1]);
                w4[e] = *reinterpret_cast<uint32_t*>(&h);
            }
            *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(dst) + c * 256 + lane * 8) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
        }
    }
}

// The "database" entry of the dynamic bit-width problem (Section 5, "Measuring Grid Parameters"): the layer's relative
// quantisation error t^2 = ||W^ - W||_F^2 / ||W||_F^2, accumulated as the two sums without materialising W^.
template <int P, typename T>
__global__ void __launch_bounds__(256) layer_error_kernel(const uint8_t* __restrict__ canonical, const __half* __restrict__ scales,
                                                          const float* __restrict__ grid, const T* __restrict__ W,
                                                          int64_t N, int64_t K, uint64_t xi, double* __restrict__ sums) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t groups = K / kGroup;
    if (warp >= N * groups) return;
    const int64_t row = warp / groups, gi = warp % groups;
    float v[32];
    dequantize_group<P>(canonical, scales, grid, K, xi, row, gi, lane, v);
    const T* src = W + row * K + gi * kGroup;
    float num = 0.f, den = 0.f;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const float w = (float)src[c * 256 + lane * 8 + e];
            const float dlt = v[c * 8 + e] - w;
            num = fmaf(dlt, dlt, num);
            den = fmaf(w, w, den);
        }
    }
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) {
        num += __shfl_xor_sync(0xffffffffu, num, m);
        den += __shfl_xor_sync(0xffffffffu, den, m);
    }
    if (lane == 0) {
        atomicAdd(sums, (double)num);
        atomicAdd(sums + 1, (double)den);
    }
}

}  // namespace

int launch_layer_error(const higgs_desc& d, const uint8_t* canonical, const void* scales, const float* grid, const void* W,
                       int w_dtype, double* sums, cudaStream_t st) {
    if (cudaMemsetAsync(sums, 0, 2 * sizeof(double), st) != cudaSuccess) return HIGGS_ERR_CUDA;
    const int64_t warps = d.N * (d.K / kGroup);
    if (warps == 0) return HIGGS_OK;
    const unsigned blocks = (unsigned)((warps + 7) / 8);
    const __half* sc = static_cast<const __half*>(scales);
    if (d.p == 2 && w_dtype == HIGGS_F32)
        layer_error_kernel<2, float><<<blocks, 256, 0, st>>>(canonical, sc, grid, static_cast<const float*>(W), d.N, d.K, d.rht_seed, sums);
    else if (d.p == 2 && w_dtype == HIGGS_BF16)
        layer_error_kernel<2, __nv_bfloat16><<<blocks, 256, 0, st>>>(canonical, sc, grid, static_cast<const __nv_bfloat16*>(W), d.N, d.K, d.rht_seed, sums);
    else if (d.p == 1 && w_dtype == HIGGS_F32)
        layer_error_kernel<1, float><<<blocks, 256, 0, st>>>(canonical, sc, grid, static_cast<const float*>(W), d.N, d.K, d.rht_seed, sums);
    else if (d.p == 1 && w_dtype == HIGGS_BF16)
        layer_error_kernel<1, __nv_bfloat16><<<blocks, 256, 0, st>>>(canonical, sc, grid, static_cast<const __nv_bfloat16*>(W), d.N, d.K, d.rht_seed, sums);
    else
        return HIGGS_ERR_UNSUPPORTED;
    return cuda_status(cudaGetLastError());
}

int launch_dequantize(const higgs_desc& d, const uint8_t* canonical, const void* scales, const float* grid, void* W_out,
                      int w_dtype, cudaStream_t st) {
    const int64_t warps = d.N * (d.K / kGroup);
    if (warps == 0) return HIGGS_OK;
    const unsigned blocks = (unsigned)((warps + 7) / 8);
    const __half* sc = static_cast<const __half*>(scales);
    if (d.p == 2 && w_dtype == HIGGS_F32)
        dequantize_kernel<2, float><<<blocks, 256, 0, st>>>(canonical, sc, grid, static_cast<float*>(W_out), d.N, d.K, d.rht_seed);
    else if (d.p == 2 && w_dtype == HIGGS_BF16)
        dequantize_kernel<2, __nv_bfloat16><<<blocks, 256, 0, st>>>(canonical, sc, grid, static_cast<__nv_bfloat16*>(W_out), d.N, d.K, d.rht_seed);
    else if (d.p == 1 && w_dtype == HIGGS_F32)
        dequantize_kernel<1, float><<<blocks, 256, 0, st>>>(canonical, sc, grid, static_cast<float*>(W_out), d.N, d.K, d.rht_seed);
    else if (d.p == 1 && w_dtype == HIGGS_BF16)
        dequantize_kernel<1, __nv_bfloat16><<<blocks, 256, 0, st>>>(canonical, sc, grid, static_cast<__nv_bfloat16*>(W_out), d.N, d.K, d.rht_seed);
    else
        return HIGGS_ERR_UNSUPPORTED;
    return cuda_status(cudaGetLastError());
}

}  // namespace higgs
