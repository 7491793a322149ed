// Encoder of Algorithm 1 for any grid (1 <= p <= 4, n <= 4096, n need not be a power of two): the grids the paper
// evaluates beside the kernel-supported ones, e.g. (p, n) = (3, 830), (2, 88), (2, 361), (1, 19) ("Experiment
// Configurations").  It emits one 16-bit code per tuple, row-major fp16 scales and, optionally, the two sums behind
// the layer's relative error t^2 ("Proof of Expected Error"), so grids can be compared without a product kernel.
//
// Tuples: the 1024 rotated values of a group are cut into ceil(1024/p) consecutive p-tuples; when p does not divide
// 1024 the last tuple is completed with zeros and matched on all p coordinates (the paper does not say; its
// reconstruction drops the completed coordinates).
#include "common.cuh"

namespace higgs {

namespace {

template <typename T>
__device__ __forceinline__ float to_f32(T v);
template <>
__device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

constexpr int kGeneralWarps = 4;

// One warp per (row, group).  Steps in the order of Algorithm 1; the rotated group goes through shared memory so that
// lane l can pick up tuples l, l + 32, ... whatever p is; the grid ([n][P] floats, P padded to PS) is scanned once
// per warp with every grid point compared against all of the lane's tuples.  fp32 distances in the plain
// sum (x_k - g_k)^2 form in coordinate order, strict '<' (lowest index wins a tie).
template <typename T, int P>
__global__ void __launch_bounds__(kGeneralWarps * 32) encode_general_kernel(
    const T* __restrict__ W, const float* __restrict__ grid, int n, uint16_t* __restrict__ codes,
    __half* __restrict__ scales, double* __restrict__ sums, int64_t N, int64_t K, uint64_t xi) {
    constexpr int PS = P == 3 ? 4 : P;                       // shared-memory stride of a grid point
    constexpr int kTuples = (kGroup + P - 1) / P;            // per group
    constexpr int kPerLane = (kTuples + 31) / 32;
    extern __shared__ __align__(16) float gen_smem[];
    float* sgrid = gen_smem;                                  // [n][PS]
    float* srot = gen_smem + (size_t)n * PS;                  // [warps][1024 + 4]

    for (int i = threadIdx.x; i < n * PS; i += blockDim.x) {
        const int c = i / PS, k = i % PS;
        sgrid[i] = k < P ? grid[c * P + k] : 0.f;
    }
    __syncthreads();

    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    float* rot = srot + wib * (kGroup + 4);
    const int64_t groups = K / kGroup;
    const int64_t total = N * groups;
    double err_acc = 0.0, nrm_acc = 0.0;

    for (int64_t item = (int64_t)blockIdx.x * kGeneralWarps + wib; item < total; item += (int64_t)gridDim.x * kGeneralWarps) {
        const int64_t row = item / groups, gi = item % groups;
        const T* src = W + row * K + gi * kGroup;
        float v[32];
#pragma unroll
        for (int r = 0; r < 32; ++r) v[r] = to_f32<T>(src[fwht_index(lane, r)]);
        float ss = 0.0f;
#pragma unroll
        for (int r = 0; r < 32; ++r) ss = fmaf(v[r], v[r], ss);
#pragma unroll
        for (int m = 16; m >= 1; m >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, m);
        const float s = sqrtf(ss);
        const float inv = s > 0.0f ? 1.0f / s : 0.0f;
#pragma unroll
        for (int r = 0; r < 32; ++r) v[r] *= inv;
        apply_signs1024(v, xi, gi * kGroup, lane);
        fwht1024_warp(v, lane);

        const __half sh = __float2half_rn(s * 0.03125f);      // s / sqrt(1024), the stored scale
        if (lane == 0) scales[row * groups + gi] = sh;

        __syncwarp();
#pragma unroll
        for (int r = 0; r < 32; ++r) rot[fwht_index(lane, r)] = v[r];
        if (lane < 4) rot[kGroup + lane] = 0.f;               // the completion of a short last tuple
        __syncwarp();

        float x[kPerLane][P];
#pragma unroll
        for (int u = 0; u < kPerLane; ++u) {
            const int t = u * 32 + lane;
#pragma unroll
            for (int k = 0; k < P; ++k) x[u][k] = t < kTuples ? rot[t * P + k] : 0.f;
        }
        float best[kPerLane];
        int bi[kPerLane];
#pragma unroll
        for (int u = 0; u < kPerLane; ++u) { best[u] = INFINITY; bi[u] = 0; }
        for (int c = 0; c < n; ++c) {
            float gp[P];
            if constexpr (P == 1) {
                gp[0] = sgrid[c];
            } else if constexpr (P == 2) {
                const float2 q = *reinterpret_cast<const float2*>(&sgrid[2 * c]);
                gp[0] = q.x; gp[1] = q.y;
            } else {
                const float4 q = *reinterpret_cast<const float4*>(&sgrid[4 * c]);
                gp[0] = q.x; gp[1] = q.y; gp[2] = q.z;
                if constexpr (P == 4) gp[3] = q.w;
            }
#pragma unroll
            for (int u = 0; u < kPerLane; ++u) {
                float d = 0.f;
#pragma unroll
                for (int k = 0; k < P; ++k) {
                    const float e = x[u][k] - gp[k];
                    d = k == 0 ? e * e : fmaf(e, e, d);
                }
                if (d < best[u]) { best[u] = d; bi[u] = c; }
            }
        }
        uint16_t* dst = codes + (row * groups + gi) * kTuples;
        float err = 0.f;                                       // || s' G[q] - (s / 32) w+ ||^2 over the group's own inputs
        const float sq = __half2float(sh), sr = s * 0.03125f;
#pragma unroll
        for (int u = 0; u < kPerLane; ++u) {
            const int t = u * 32 + lane;
            if (t < kTuples) {
                dst[t] = (uint16_t)bi[u];
#pragma unroll
                for (int k = 0; k < P; ++k)
                    if (t * P + k < kGroup) {
                        const float e = fmaf(sq, sgrid[bi[u] * PS + k], -sr * x[u][k]);
                        err = fmaf(e, e, err);
                    }
            }
        }
        if (sums) {
#pragma unroll
            for (int m = 16; m >= 1; m >>= 1) err += __shfl_xor_sync(0xffffffffu, err, m);
            err_acc += (double)err;
            nrm_acc += (double)ss;
        }
    }
    if (sums && lane == 0 && nrm_acc != 0.0) {
        atomicAdd(&sums[0], err_acc);
        atomicAdd(&sums[1], nrm_acc);
    }
}

template <typename T, int P>
int launch_p(int n, int64_t N, int64_t K, uint64_t xi, const void* W, const float* grid, uint16_t* codes, void* scales,
             double* sums, cudaStream_t st) {
    constexpr int PS = P == 3 ? 4 : P;
    const size_t smem = sizeof(float) * ((size_t)n * PS + (size_t)kGeneralWarps * (kGroup + 4));
    cudaError_t e = cudaFuncSetAttribute(encode_general_kernel<T, P>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_status(e);
    const int64_t items = N * (K / kGroup);
    int64_t blocks = (items + kGeneralWarps - 1) / kGeneralWarps;
    const int64_t cap = 148 * (smem > 100 * 1024 ? 2 : 4);      // persistent over the work when it is large
    if (blocks > cap) blocks = cap;
    encode_general_kernel<T, P><<<(unsigned)blocks, kGeneralWarps * 32, smem, st>>>(
        static_cast<const T*>(W), grid, n, codes, static_cast<__half*>(scales), sums, N, K, xi);
    return cuda_status(cudaGetLastError());
}

template <typename T>
int launch_t(int p, int n, int64_t N, int64_t K, uint64_t xi, const void* W, const float* grid, uint16_t* codes,
             void* scales, double* sums, cudaStream_t st) {
    switch (p) {
        case 1: return launch_p<T, 1>(n, N, K, xi, W, grid, codes, scales, sums, st);
        case 2: return launch_p<T, 2>(n, N, K, xi, W, grid, codes, scales, sums, st);
        case 3: return launch_p<T, 3>(n, N, K, xi, W, grid, codes, scales, sums, st);
        case 4: return launch_p<T, 4>(n, N, K, xi, W, grid, codes, scales, sums, st);
    }
    return HIGGS_ERR_UNSUPPORTED;
}

}  // namespace

int launch_encode_general(int p, int n, int64_t N, int64_t K, uint64_t xi, const void* W, int w_dtype, const float* grid,
                          uint16_t* codes, void* scales, double* sums, cudaStream_t st) {
    if (sums) {
        cudaError_t e = cudaMemsetAsync(sums, 0, 2 * sizeof(double), st);
        if (e != cudaSuccess) return cuda_status(e);
    }
    if (w_dtype == HIGGS_BF16)
        return launch_t<__nv_bfloat16>(p, n, N, K, xi, W, grid, codes, scales, sums, st);
    return launch_t<float>(p, n, N, K, xi, W, grid, codes, scales, sums, st);
}

}  // namespace higgs
