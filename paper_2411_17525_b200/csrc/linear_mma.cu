// Small-batch product in the rotated space (Appendix F, "Rotating Activations"):
//   y[b][r] = sum_i scale[r][i] * sum_t < G[code[r][i][t]], x+[b][i][2t:2t+2] >
// for B <= 16 tokens per launch.  The kernel is bound by the HBM stream of packed
// codes; every code costs one shared-memory table lookup whose 32-bit result (an
// fp16 pair = two consecutive inputs of one row) IS an A-fragment register of an
// m16n8k16 tensor-core step, so dequantisation is fused into the operand load and
// accumulation is fp32.
#include "common.cuh"

namespace higgs {

namespace {

struct LinearParams {
    const __half* xdag;    // [B][K] rotated activations, fp16
    const uint8_t* packed; // packed code stream
    const __half* scales;  // [N][K/g]
    const float* grid;     // [n][p]
    void* y;               // [B][ldy]
    int64_t N, K, ldy;
    int B;                 // valid tokens (<= 8 * NB)
    int n, p;
    int chunks;            // K is split into `chunks` ranges handled by different blocks
    int warps_per_chunk;   // = blockDim.x / 32
    int parts;             // blocks per chunk; row tiles are split evenly among them
    int y_mode;            // 0: store fp32, 1: store bf16, 2: atomicAdd fp32
};

constexpr uint32_t kLutBytes = 65536;        // 256 entries x 256-byte row (32 lanes x 4 B, upper half unused)
constexpr uint32_t kSmemBytes = 2 * kLutBytes + 2048;

__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint4 ldg_stream16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ uint2 ldg_stream8(const void* p) {
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}

// Code words of one (row tile, k-slice) for this lane.
template <int KS, bool SIX>
struct TileCodes {
    // byte-LUT: KS/64 x 16 B.  six-bit: KS/128 super-blocks x 3 planes x 8 B.
    static constexpr int kWords = SIX ? (KS / 128) * 6 : (KS / 64) * 4;
    uint32_t w[kWords];
    __device__ __forceinline__ void load(const uint8_t* __restrict__ packed, int64_t rt, int64_t kblocks, int64_t kb0,
                                         int lane) {
        if (SIX) {
#pragma unroll
            for (int sb = 0; sb < KS / 128; ++sb) {
                const int64_t base = (rt * (kblocks >> 1) + (kb0 >> 1) + sb) * 3;
#pragma unroll
                for (int pl = 0; pl < 3; ++pl) {
                    uint2 q = ldg_stream8(packed + ((base + pl) * 64 + 2 * lane) * 4);
                    w[sb * 6 + pl * 2] = q.x;
                    w[sb * 6 + pl * 2 + 1] = q.y;
                }
            }
        } else {
#pragma unroll
            for (int j = 0; j < KS / 64; ++j) {
                uint4 q = ldg_stream16(packed + ((rt * kblocks + kb0 + j) * 32 + lane) * 16);
                w[j * 4] = q.x; w[j * 4 + 1] = q.y; w[j * 4 + 2] = q.z; w[j * 4 + 3] = q.w;
            }
        }
    }
    // four byte-aligned table indices (slots 4m..4m+3) of 64-input block j, step m
    __device__ __forceinline__ uint32_t index_word(int j, int m) const {
        if (!SIX) return w[j * 4 + m];
        const int sb = j >> 1, h = j & 1;
        const uint32_t lo = w[sb * 6 + (m >> 1) * 2 + h];
        const uint32_t hi = w[sb * 6 + 4 + h];
        const uint32_t a = (m & 1) ? (lo >> 4) : lo;
        const uint32_t b = (m == 0) ? (hi << 4) : (m == 1) ? (hi << 2) : (m == 2) ? hi : (hi >> 2);
        // (a & 0x0f0f0f0f) | (b & 0xf0f0f0f0): bits 6-7 of each byte are don't-care (table is replicated)
        uint32_t r;
        asm("lop3.b32 %0, %1, %2, 0x0f0f0f0f, 0xe4;" : "=r"(r) : "r"(a), "r"(b));
        return r;
    }
};

template <int NB, int KS, bool SIX>
__global__ void __launch_bounds__(512, 1) linear_mma_kernel(const LinearParams prm) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;

    // ---- shared memory carve-up: 64 KB-aligned table + reduction scratch ----
    const uint32_t smem_base = (uint32_t)__cvta_generic_to_shared(smem_raw);
    const uint32_t lut_addr = (smem_base + 0xffffu) & ~0xffffu;
    uint8_t* lut_ptr = smem_raw + (lut_addr - smem_base);
    // scratch goes in whichever side of the table has >= 33 KB free
    float* red = reinterpret_cast<float*>((lut_addr - smem_base >= 33 * 1024) ? smem_raw : lut_ptr + kLutBytes);

    // ---- table: entry(idx) replicated once per lane (bank = lane): conflict-free ----
    {
        const int n = prm.n, p = prm.p;
        for (int i = tid; i < 256 * 32; i += blockDim.x) {
            const int idx = i >> 5, l = i & 31;
            float lo, hi;
            if (p == 2) {
                const int c = idx & (n - 1);
                lo = __ldg(prm.grid + 2 * c);
                hi = __ldg(prm.grid + 2 * c + 1);
            } else {
                lo = __ldg(prm.grid + (idx & 15));
                hi = __ldg(prm.grid + (idx >> 4));
            }
            __half2 h = __floats2half2_rn(lo, hi);
            *reinterpret_cast<uint32_t*>(lut_ptr + idx * 256 + l * 4) = *reinterpret_cast<uint32_t*>(&h);
        }
    }

    const int chunk = blockIdx.x % prm.chunks;
    const int part = blockIdx.x / prm.chunks;
    const int64_t tiles = prm.N / kRowTile;
    const int64_t rt_begin = tiles * part / prm.parts, rt_end = tiles * (part + 1) / prm.parts;
    const int64_t kblocks = prm.K / kBlockK;
    const int64_t groups = prm.K / kGroup;
    const int64_t k0 = ((int64_t)chunk * prm.warps_per_chunk + warp) * KS;
    const int64_t kb0 = k0 / kBlockK;
    const int64_t gi = k0 / kGroup;

    // ---- B fragments of this warp's k-slice stay in registers for the whole kernel ----
    uint32_t bfrag[KS / 16][NB][2];
#pragma unroll
    for (int s = 0; s < KS / 16; ++s) {
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
            const int col = nb * 8 + g;
            uint32_t b0 = 0u, b1 = 0u;
            if (col < prm.B) {
                const __half* src = prm.xdag + (int64_t)col * prm.K + k0 + s * 16 + 2 * t;
                b0 = *reinterpret_cast<const uint32_t*>(src);
                b1 = *reinterpret_cast<const uint32_t*>(src + 8);
            }
            bfrag[s][nb][0] = b0;
            bfrag[s][nb][1] = b1;
        }
    }
    __syncthreads();

    const uint32_t lut_lane = lut_addr + lane * 4;
    const int nwarps = blockDim.x >> 5;
    constexpr int kCols = 8 * NB;
    constexpr int kRedTile = 16 * kCols;   // floats per warp per buffer

    TileCodes<KS, SIX> cur, nxt;
    float s_lo = 0.f, s_hi = 0.f, ns_lo = 0.f, ns_hi = 0.f;
    if (rt_begin < rt_end) {
        cur.load(prm.packed, rt_begin, kblocks, kb0, lane);
        s_lo = __half2float(prm.scales[(rt_begin * 16 + g) * groups + gi]);
        s_hi = __half2float(prm.scales[(rt_begin * 16 + g + 8) * groups + gi]);
    }
    int buf = 0;
    for (int64_t rt = rt_begin; rt < rt_end; ++rt) {
        if (rt + 1 < rt_end) {
            nxt.load(prm.packed, rt + 1, kblocks, kb0, lane);
            ns_lo = __half2float(prm.scales[((rt + 1) * 16 + g) * groups + gi]);
            ns_hi = __half2float(prm.scales[((rt + 1) * 16 + g + 8) * groups + gi]);
        }
        float acc[NB][4];
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) acc[nb][0] = acc[nb][1] = acc[nb][2] = acc[nb][3] = 0.f;
#pragma unroll
        for (int j = 0; j < KS / 64; ++j) {
#pragma unroll
            for (int m = 0; m < 4; ++m) {
                const uint32_t iw = cur.index_word(j, m);
                const uint32_t a0 = lds32(__byte_perm(iw, lut_lane, 0x7604));
                const uint32_t a1 = lds32(__byte_perm(iw, lut_lane, 0x7614));
                const uint32_t a2 = lds32(__byte_perm(iw, lut_lane, 0x7624));
                const uint32_t a3 = lds32(__byte_perm(iw, lut_lane, 0x7634));
#pragma unroll
                for (int nb = 0; nb < NB; ++nb)
                    mma16816(acc[nb], a0, a1, a2, a3, bfrag[j * 4 + m][nb][0], bfrag[j * 4 + m][nb][1]);
            }
        }
        // scale (fp32) and reduce over the warps of this block; layout [warp][col][row]
        float* mine = red + buf * (nwarps * kRedTile) + warp * kRedTile;
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
            mine[(nb * 8 + 2 * t) * 16 + g] = acc[nb][0] * s_lo;
            mine[(nb * 8 + 2 * t + 1) * 16 + g] = acc[nb][1] * s_lo;
            mine[(nb * 8 + 2 * t) * 16 + g + 8] = acc[nb][2] * s_hi;
            mine[(nb * 8 + 2 * t + 1) * 16 + g + 8] = acc[nb][3] * s_hi;
        }
        __syncthreads();
        if (tid < kRedTile) {
            const int col = tid >> 4, r = tid & 15;
            if (col < prm.B) {
                const float* src = red + buf * (nwarps * kRedTile) + tid;
                float sum = 0.f;
                for (int w = 0; w < nwarps; ++w) sum += src[w * kRedTile];
                const int64_t o = (int64_t)col * prm.ldy + rt * 16 + r;
                if (prm.y_mode == 0) static_cast<float*>(prm.y)[o] = sum;
                else if (prm.y_mode == 1) static_cast<__nv_bfloat16*>(prm.y)[o] = __float2bfloat16_rn(sum);
                else atomicAdd(static_cast<float*>(prm.y) + o, sum);
            }
        }
        buf ^= 1;
        cur = nxt;
        s_lo = ns_lo;
        s_hi = ns_hi;
    }
}

__global__ void convert_out_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, size_t count) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) dst[i] = __float2bfloat16_rn(src[i]);
}

int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
        cached[dev] = v;
    }
    return cached[dev];
}

struct Plan {
    int nb, ks, chunks, warps_per_chunk, parts;
};

Plan make_plan(const higgs_desc& d, int64_t B) {
    Plan pl;
    const bool six = format_of(d.p, d.n) == Format::kSixBit;
    pl.nb = B <= 8 ? 1 : 2;
    const int ks_min = six ? 128 : 64;
    pl.ks = 256 / pl.nb;
    while (d.K / pl.ks < 16 && pl.ks > ks_min) pl.ks /= 2;
    const int slices = (int)(d.K / pl.ks);
    pl.chunks = (slices + 15) / 16;
    while (slices % pl.chunks) ++pl.chunks;
    pl.warps_per_chunk = slices / pl.chunks;
    const int64_t tiles = d.N / kRowTile;
    int64_t parts = sm_count() / pl.chunks;
    if (parts < 1) parts = 1;
    if (parts > tiles) parts = tiles;
    pl.parts = (int)parts;
    return pl;
}

template <int NB, int KS, bool SIX>
int launch_one(const LinearParams& prm, cudaStream_t st) {
    static bool configured[64] = {false};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(linear_mma_kernel<NB, KS, SIX>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)kSmemBytes);
        if (e != cudaSuccess) return HIGGS_ERR_CUDA;
        configured[dev] = true;
    }
    linear_mma_kernel<NB, KS, SIX>
        <<<(unsigned)(prm.chunks * prm.parts), (unsigned)(prm.warps_per_chunk * 32), kSmemBytes, st>>>(prm);
    return cuda_status(cudaGetLastError());
}

}  // namespace

int linear_k_chunks(const higgs_desc& d, int64_t B) { return make_plan(d, B > 16 ? 16 : B).chunks; }

// y_mode as in LinearParams.  B <= 16.
int launch_linear_mma(const higgs_desc& d, const __half* xdag, int64_t B, const void* packed, const void* scales,
                      const float* grid, void* y, int64_t ldy, int y_mode, cudaStream_t st) {
    if (d.N == 0) return HIGGS_OK;
    const Plan pl = make_plan(d, B);
    LinearParams prm;
    prm.xdag = xdag;
    prm.packed = static_cast<const uint8_t*>(packed);
    prm.scales = static_cast<const __half*>(scales);
    prm.grid = grid;
    prm.y = y;
    prm.N = d.N; prm.K = d.K; prm.ldy = ldy;
    prm.B = (int)B;
    prm.n = d.n; prm.p = d.p;
    prm.chunks = pl.chunks;
    prm.warps_per_chunk = pl.warps_per_chunk;
    prm.parts = pl.parts;
    prm.y_mode = y_mode;
    const bool six = format_of(d.p, d.n) == Format::kSixBit;
#define HIGGS_LAUNCH(NB_, KS_, SIX_) \
    if (pl.nb == NB_ && pl.ks == KS_ && six == SIX_) return launch_one<NB_, KS_, SIX_>(prm, st)
    HIGGS_LAUNCH(1, 256, false);
    HIGGS_LAUNCH(1, 128, false);
    HIGGS_LAUNCH(1, 64, false);
    HIGGS_LAUNCH(2, 128, false);
    HIGGS_LAUNCH(2, 64, false);
    HIGGS_LAUNCH(1, 256, true);
    HIGGS_LAUNCH(1, 128, true);
    HIGGS_LAUNCH(2, 128, true);
#undef HIGGS_LAUNCH
    return HIGGS_ERR_UNSUPPORTED;
}

int launch_convert_out(const float* y32, void* y, int y_dtype, size_t count, cudaStream_t st) {
    if (y_dtype != HIGGS_BF16) return HIGGS_ERR_UNSUPPORTED;
    if (count == 0) return HIGGS_OK;
    convert_out_kernel<<<(unsigned)((count + 255) / 256), 256, 0, st>>>(y32, static_cast<__nv_bfloat16*>(y), count);
    return cuda_status(cudaGetLastError());
}

}  // namespace higgs
