// Grid fit of Algorithm 2 ("CLVQ(n, p), computed once"), run as Lloyd's batch
// iteration on caller-provided samples of N(0, I_p): the assignment step is the
// encoder's exhaustive nearest-point search, the update a segmented mean.
#include "common.cuh"

namespace higgs {

namespace {

struct GridWs {
    float* centres;               // [n][p]
    double* sums;                 // [n][p]
    unsigned long long* counts;   // [n]
    int32_t* assign;              // [m]
    double* err;                  // [2]: running, last completed
    int32_t* flags;               // [0] changed, [1] done, [2] iterations, [3] grid-barrier arrivals (persistent fit)
};

__host__ __device__ inline size_t up256(size_t v) { return (v + 255) / 256 * 256; }

GridWs carve(void* ws, int p, int n, int64_t m) {
    uint8_t* b = static_cast<uint8_t*>(ws);
    GridWs w;
    w.centres = reinterpret_cast<float*>(b); b += up256(sizeof(float) * n * p);
    w.sums = reinterpret_cast<double*>(b); b += up256(sizeof(double) * n * p);
    w.counts = reinterpret_cast<unsigned long long*>(b); b += up256(sizeof(unsigned long long) * n);
    w.err = reinterpret_cast<double*>(b); b += 256;
    w.flags = reinterpret_cast<int32_t*>(b); b += 256;
    w.assign = reinterpret_cast<int32_t*>(b);
    (void)m;
    return w;
}

__global__ void grid_init_kernel(GridWs w, const float* __restrict__ samples, int p, int n, int64_t m) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < m) w.assign[i] = -1;
    if (i < (int64_t)n * p) { w.centres[i] = samples[i]; w.sums[i] = 0.0; }
    if (i < n) w.counts[i] = 0ull;
    if (i < 2) w.err[i] = 0.0;
    if (i < 8) w.flags[i] = 0;
}

// Assignment step.  The centres sit in dynamic shared memory ([n][P] floats, at most 64 KB).  SMALL (n <= 256): the
// per-cell sums are first collected in shared memory and then added to the global ones; otherwise every sample adds
// to the global sums directly (with thousands of cells the atomics rarely collide).  Distances are the plain
// sum of (x_k - c_k)^2 in coordinate order, fp32, strict '<' (lowest index wins a tie) - the encoder's rule.
template <int P, bool SMALL>
__device__ __forceinline__ void assign_body(const GridWs& w, const float* __restrict__ samples, int n, int64_t m,
                                            unsigned char* grid_smem) {
    float* sc = reinterpret_cast<float*>(grid_smem);
    double* ssum = reinterpret_cast<double*>(grid_smem + up256(sizeof(float) * n * P));
    unsigned int* scnt = reinterpret_cast<unsigned int*>(ssum + (SMALL ? n * P : 0));
    __shared__ double serr;
    __shared__ int schanged;
    for (int i = threadIdx.x; i < n * P; i += blockDim.x) {
        sc[i] = __ldcg(&w.centres[i]);       // (bypasses L1: in the persistent fit another block rewrote the centres)
        if (SMALL) ssum[i] = 0.0;
    }
    if (SMALL)
        for (int i = threadIdx.x; i < n; i += blockDim.x) scnt[i] = 0u;
    if (threadIdx.x == 0) { serr = 0.0; schanged = 0; }
    __syncthreads();
    double err = 0.0;
    int changed = 0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < m; i += (int64_t)gridDim.x * blockDim.x) {
        float x[P];
#pragma unroll
        for (int k = 0; k < P; ++k) x[k] = samples[i * P + k];
        float best = INFINITY;
        int bi = 0;
        for (int c = 0; c < n; ++c) {
            float d = 0.f;
#pragma unroll
            for (int k = 0; k < P; ++k) {
                const float e = x[k] - sc[c * P + k];
                d = k == 0 ? e * e : fmaf(e, e, d);
            }
            if (d < best) { best = d; bi = c; }
        }
        if (w.assign[i] != bi) { w.assign[i] = bi; ++changed; }
        err += (double)best;
        if (SMALL) {
#pragma unroll
            for (int k = 0; k < P; ++k) atomicAdd(&ssum[bi * P + k], (double)x[k]);
            atomicAdd(&scnt[bi], 1u);
        } else {
#pragma unroll
            for (int k = 0; k < P; ++k) atomicAdd(&w.sums[bi * P + k], (double)x[k]);
            atomicAdd(&w.counts[bi], 1ull);
        }
    }
    atomicAdd(&serr, err);
    if (changed) atomicAdd(&schanged, changed);
    __syncthreads();
    if (SMALL) {
        for (int i = threadIdx.x; i < n * P; i += blockDim.x)
            if (ssum[i] != 0.0) atomicAdd(&w.sums[i], ssum[i]);
        for (int i = threadIdx.x; i < n; i += blockDim.x)
            if (scnt[i]) atomicAdd(&w.counts[i], (unsigned long long)scnt[i]);
    }
    if (threadIdx.x == 0) {
        atomicAdd(&w.err[0], serr);
        if (schanged) atomicAdd(&w.flags[0], schanged);
    }
}

template <int P, bool SMALL>
__global__ void __launch_bounds__(256) grid_assign_kernel(GridWs w, const float* __restrict__ samples, int n, int64_t m) {
    extern __shared__ __align__(16) unsigned char grid_smem[];
    if (w.flags[1]) return;
    assign_body<P, SMALL>(w, samples, n, m, grid_smem);
}

__device__ __forceinline__ void update_body(const GridWs& w, int p, int n) {
    const int changed = __ldcg(&w.flags[0]);
    __syncthreads();
    for (int i = threadIdx.x; i < n * p; i += blockDim.x) {
        const unsigned long long cnt = __ldcg(&w.counts[i / p]);
        if (changed && cnt) w.centres[i] = (float)(__ldcg(&w.sums[i]) / (double)cnt);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < n * p; i += blockDim.x) w.sums[i] = 0.0;
    for (int i = threadIdx.x; i < n; i += blockDim.x) w.counts[i] = 0ull;
    if (threadIdx.x == 0) {
        w.err[1] = __ldcg(&w.err[0]);
        w.err[0] = 0.0;
        w.flags[2] = __ldcg(&w.flags[2]) + 1;
        w.flags[0] = 0;
        if (!changed) w.flags[1] = 1;
    }
}

__global__ void grid_update_kernel(GridWs w, int p, int n) {
    if (w.flags[1]) return;
    update_body(w, p, n);
}

// ---- the whole iteration in ONE cooperatively launched kernel ---------------------------------------------------
// Every block is resident (the launch fails otherwise), so the blocks can meet at a barrier between the assignment and
// the update step: a counter in the workspace that every block's first thread increments and then polls, with a limit
// on the polls - a barrier that runs out raises the grid-fit status word and every block leaves.
__device__ int g_grid_status = 0;
constexpr unsigned kGridBarrierLimit = 1u << 22;

__device__ __forceinline__ bool grid_barrier(int32_t* counter, int target) {
    __syncthreads();
    int ok = 1;
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(counter, 1);
        unsigned it = 0;
        for (;;) {
            int v;
            asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
            if (v >= target) break;
            if (++it > kGridBarrierLimit) { ok = 0; atomicExch(&g_grid_status, (int)HIGGS_ERR_TIMEOUT); break; }
            __nanosleep(64);
        }
        __threadfence();
    }
    return __syncthreads_and(ok) != 0;
}

template <int P, bool SMALL>
__global__ void __launch_bounds__(256) grid_fit_kernel(GridWs w, const float* __restrict__ samples, int n, int64_t m, int max_iters) {
    extern __shared__ __align__(16) unsigned char grid_smem[];
    const int blocks = (int)gridDim.x;
    int barrier_no = 0;
    for (int it = 0; it < max_iters; ++it) {
        assign_body<P, SMALL>(w, samples, n, m, grid_smem);
        if (!grid_barrier(&w.flags[3], ++barrier_no * blocks)) return;
        if (blockIdx.x == 0) update_body(w, P, n);
        if (!grid_barrier(&w.flags[3], ++barrier_no * blocks)) return;
        if (*reinterpret_cast<volatile int32_t*>(&w.flags[1])) return;       // no assignment changed: a fixed point
    }
}

__global__ void grid_finalize_kernel(GridWs w, int p, int n, int64_t m, float* __restrict__ grid_out,
                                     float* __restrict__ mse_out, int32_t* __restrict__ iters_out) {
    // lexicographic sort by rank counting (coordinate 0 first; equal points keep their index order)
    for (int c = threadIdx.x; c < n; c += blockDim.x) {
        int rank = 0;
        for (int o = 0; o < n; ++o) {
            int cmp = 0;                                   // sign of (centre o) - (centre c)
            for (int k = 0; k < p && cmp == 0; ++k) {
                const float a = w.centres[c * p + k], b = w.centres[o * p + k];
                cmp = b < a ? -1 : (b > a ? 1 : 0);
            }
            rank += (cmp < 0 || (cmp == 0 && o < c)) ? 1 : 0;
        }
        for (int k = 0; k < p; ++k) grid_out[rank * p + k] = w.centres[c * p + k];
    }
    if (threadIdx.x == 0) {
        if (mse_out) *mse_out = (float)(w.err[1] / ((double)m * p));
        if (iters_out) *iters_out = w.flags[1] ? w.flags[2] : -w.flags[2];
    }
}

// ---- constrained (uniform) grid, Section 4.3 "Constrained HIGGS" ------------------------------------------
// n equally spaced levels (k - (n-1)/2) * step, symmetric about 0 (the Gaussian is); the step minimises the expected
// squared error of rounding N(0,1):  MSE(step) = sum over cells of  M2 - 2 c M1 + c^2 P  with the cell's probability
// P, first moment M1 = phi(a) - phi(b) and second moment M2 = P + a phi(a) - b phi(b)  (a, b the cell's thresholds,
// the outer cells unbounded).  One block; thread i owns cell i; golden-section search on the step in fp64.
__device__ __forceinline__ double d_phi(double x) { return 0.3989422804014327 * exp(-0.5 * x * x); }
__device__ __forceinline__ double d_Phi(double x) { return 0.5 * erfc(-x * 0.7071067811865476); }

__device__ double uniform_mse_block(int n, double step, double* red) {
    double term = 0.0;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const double c = ((double)i - 0.5 * (double)(n - 1)) * step;
        const bool lo_inf = i == 0, hi_inf = i == n - 1;
        const double a = c - 0.5 * step, b = c + 0.5 * step;
        const double Pa = lo_inf ? 0.0 : d_Phi(a), Pb = hi_inf ? 1.0 : d_Phi(b);
        const double fa = lo_inf ? 0.0 : d_phi(a), fb = hi_inf ? 0.0 : d_phi(b);
        const double P = Pb - Pa, M1 = fa - fb, M2 = P + (lo_inf ? 0.0 : a * fa) - (hi_inf ? 0.0 : b * fb);
        term += M2 - 2.0 * c * M1 + c * c * P;
    }
    red[threadIdx.x] = term;
    __syncthreads();
    for (int s = blockDim.x / 2; s > 0; s >>= 1) {
        if ((int)threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
        __syncthreads();
    }
    const double v = red[0];
    __syncthreads();
    return v;
}

__global__ void __launch_bounds__(256) uniform_grid_kernel(int n, float* __restrict__ grid_out, float* __restrict__ step_out,
                                                           float* __restrict__ mse_out) {
    __shared__ double red[256];
    double lo = 1e-4, hi = 8.0 / n + 2.0;
    const double r = 0.6180339887498949;
    double a = hi - r * (hi - lo), b = lo + r * (hi - lo);
    double fa = uniform_mse_block(n, a, red), fb = uniform_mse_block(n, b, red);
    for (int it = 0; it < 120; ++it) {         // every thread follows the same path: the values are block-uniform
        if (fa < fb) {
            hi = b; b = a; fb = fa;
            a = hi - r * (hi - lo);
            fa = uniform_mse_block(n, a, red);
        } else {
            lo = a; a = b; fa = fb;
            b = lo + r * (hi - lo);
            fb = uniform_mse_block(n, b, red);
        }
    }
    const double step = 0.5 * (lo + hi);
    const double mse = uniform_mse_block(n, step, red);
    for (int i = threadIdx.x; i < n; i += blockDim.x) grid_out[i] = (float)(((double)i - 0.5 * (double)(n - 1)) * step);
    if (threadIdx.x == 0) {
        if (step_out) *step_out = (float)step;
        if (mse_out) *mse_out = (float)mse;
    }
}

}  // namespace

int launch_uniform_grid(int n, float* grid_out, float* step_out, float* mse_out, cudaStream_t st) {
    uniform_grid_kernel<<<1, 256, 0, st>>>(n, grid_out, step_out, mse_out);
    return cuda_status(cudaGetLastError());
}

size_t make_grid_workspace(int p, int n, int64_t m) {
    return up256(sizeof(float) * n * p) + up256(sizeof(double) * n * p) + up256(sizeof(unsigned long long) * n) + 512 +
           up256(sizeof(int32_t) * (size_t)m);
}

template <int P, bool SMALL>
static int assign_step(GridWs w, const float* samples, int n, int64_t m, unsigned blocks, cudaStream_t st) {
    const size_t smem = up256(sizeof(float) * n * P) + (SMALL ? sizeof(double) * n * P + sizeof(unsigned int) * n : 0);
    if (smem > 48 * 1024) {
        static int opted[64] = {0};                        // per instantiation and device: 1 = done, -1 = failed
        const int ok = device_once(opted, [] {
            return cudaFuncSetAttribute(grid_assign_kernel<P, SMALL>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)(up256(sizeof(float) * kMaxGridPoints * P))) == cudaSuccess ? 1 : -1;
        });
        if (ok < 0) return HIGGS_ERR_CUDA;
    }
    grid_assign_kernel<P, SMALL><<<blocks, 256, smem, st>>>(w, samples, n, m);
    return HIGGS_OK;
}

// One cooperative launch for the whole iteration; returns HIGGS_ERR_UNSUPPORTED when the device or the shape does not
// allow it (the caller then enqueues one pair of kernels per iteration).
static int sm_count_of_device() {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v < 1) v = 1;
    return v;
}

template <int P, bool SMALL>
static int fit_persistent(GridWs w, const float* samples, int n, int64_t m, int max_iters, cudaStream_t st) {
    const size_t smem = up256(sizeof(float) * n * P) + (SMALL ? sizeof(double) * n * P + sizeof(unsigned int) * n : 0);
    static int per_sm[64] = {0};          // resident blocks per SM at the largest shared-memory size, -1 = not available
    const int bps = device_once(per_sm, [] {
        int dev = 0, coop = 0, v = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop)
            return -1;
        const size_t max_smem = up256(sizeof(float) * kMaxGridPoints * P) + (SMALL ? (sizeof(double) * P + sizeof(unsigned int)) * 256 : 0);
        if (cudaFuncSetAttribute(grid_fit_kernel<P, SMALL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem) != cudaSuccess) return -1;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&v, grid_fit_kernel<P, SMALL>, 256, max_smem) != cudaSuccess || v < 1) return -1;
        return v;
    });
    if (bps < 1) return HIGGS_ERR_UNSUPPORTED;
    int64_t blocks = (m + 255) / 256;
    const int64_t cap = (int64_t)bps * sm_count_of_device();
    if (blocks > cap) blocks = cap;
    if (blocks > 592) blocks = 592;
    void* args[] = {&w, &samples, &n, &m, &max_iters};
    const cudaError_t e = cudaLaunchCooperativeKernel((const void*)grid_fit_kernel<P, SMALL>, dim3((unsigned)blocks), dim3(256), args, smem, st);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return HIGGS_ERR_UNSUPPORTED; }
    return HIGGS_OK;
}

int launch_make_grid(int p, int n, const float* samples, int64_t m, int max_iters, float* grid_out, float* mse_out,
                     int32_t* iters_out, void* ws, cudaStream_t st) {
    GridWs w = carve(ws, p, n, m);
    const int64_t init_threads = m > (int64_t)n * p ? m : (int64_t)n * p;
    grid_init_kernel<<<(unsigned)((init_threads + 255) / 256), 256, 0, st>>>(w, samples, p, n, m);
    int64_t blocks = (m + 255) / 256;
    if (blocks > 592) blocks = 592;
    const bool small = n <= 256;
    {
        int rc = HIGGS_ERR_UNSUPPORTED;
        switch (p * 2 + (small ? 1 : 0)) {
            case 3: rc = fit_persistent<1, true>(w, samples, n, m, max_iters, st); break;
            case 2: rc = fit_persistent<1, false>(w, samples, n, m, max_iters, st); break;
            case 5: rc = fit_persistent<2, true>(w, samples, n, m, max_iters, st); break;
            case 4: rc = fit_persistent<2, false>(w, samples, n, m, max_iters, st); break;
            case 7: rc = fit_persistent<3, true>(w, samples, n, m, max_iters, st); break;
            case 6: rc = fit_persistent<3, false>(w, samples, n, m, max_iters, st); break;
            case 9: rc = fit_persistent<4, true>(w, samples, n, m, max_iters, st); break;
            case 8: rc = fit_persistent<4, false>(w, samples, n, m, max_iters, st); break;
            default: return HIGGS_ERR_UNSUPPORTED;
        }
        if (rc == HIGGS_OK) {
            grid_finalize_kernel<<<1, 256, 0, st>>>(w, p, n, m, grid_out, mse_out, iters_out);
            return cuda_status(cudaGetLastError());
        }
    }
    for (int it = 0; it < max_iters; ++it) {
        int rc;
        switch (p * 2 + (small ? 1 : 0)) {
            case 3: rc = assign_step<1, true>(w, samples, n, m, (unsigned)blocks, st); break;
            case 2: rc = assign_step<1, false>(w, samples, n, m, (unsigned)blocks, st); break;
            case 5: rc = assign_step<2, true>(w, samples, n, m, (unsigned)blocks, st); break;
            case 4: rc = assign_step<2, false>(w, samples, n, m, (unsigned)blocks, st); break;
            case 7: rc = assign_step<3, true>(w, samples, n, m, (unsigned)blocks, st); break;
            case 6: rc = assign_step<3, false>(w, samples, n, m, (unsigned)blocks, st); break;
            case 9: rc = assign_step<4, true>(w, samples, n, m, (unsigned)blocks, st); break;
            case 8: rc = assign_step<4, false>(w, samples, n, m, (unsigned)blocks, st); break;
            default: return HIGGS_ERR_UNSUPPORTED;
        }
        if (rc != HIGGS_OK) return rc;
        grid_update_kernel<<<1, 256, 0, st>>>(w, p, n);
    }
    grid_finalize_kernel<<<1, 256, 0, st>>>(w, p, n, m, grid_out, mse_out, iters_out);
    return cuda_status(cudaGetLastError());
}

int read_grid_status(int clear) {
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_grid_status, sizeof(int)) != cudaSuccess) return HIGGS_ERR_CUDA;
    if (clear && v != 0) {
        const int zero = 0;
        if (cudaMemcpyToSymbol(g_grid_status, &zero, sizeof(int)) != cudaSuccess) return HIGGS_ERR_CUDA;
    }
    return v;
}

}  // namespace higgs
