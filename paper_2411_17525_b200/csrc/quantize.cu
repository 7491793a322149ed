// Encoder of Algorithm 1 (RHT-VQ): group norm, randomised Hadamard transform,
// exhaustive nearest-grid-point search, canonical codes and fp16 scales; plus the
// conversion between canonical codes and the packed, kernel-native code stream.
#include "common.cuh"

namespace higgs {

namespace {

template <typename T>
__device__ __forceinline__ void load32(const T* __restrict__ src, int lane, float (&v)[32]);

template <>
__device__ __forceinline__ void load32<__nv_bfloat16>(const __nv_bfloat16* __restrict__ src, int lane, float (&v)[32]) {
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
__device__ __forceinline__ void load32<float>(const float* __restrict__ src, int lane, float (&v)[32]) {
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        float4 a = __ldg(reinterpret_cast<const float4*>(src + c * 256 + lane * 8));
        float4 b = __ldg(reinterpret_cast<const float4*>(src + c * 256 + lane * 8 + 4));
        v[c * 8 + 0] = a.x; v[c * 8 + 1] = a.y; v[c * 8 + 2] = a.z; v[c * 8 + 3] = a.w;
        v[c * 8 + 4] = b.x; v[c * 8 + 5] = b.y; v[c * 8 + 6] = b.z; v[c * 8 + 7] = b.w;
    }
}

// One warp per (row, group).  Steps in the order of Algorithm 1:
//   s = ||w||_2 ; w+ = H diag(sign) (w/s) ; code = argmin_c ||w+_t - G[c]||^2 ; scale = s/sqrt(g).
// Distances are fp32 in the plain (x-g)^2 form; '<' keeps the lowest index on ties.
template <typename T, int P>
__global__ void __launch_bounds__(128) encode_kernel(const T* __restrict__ W, const float* __restrict__ grid, int n,
                                                     uint8_t* __restrict__ canonical, __half* __restrict__ scales,
                                                     int64_t N, int64_t K, uint64_t xi) {
    __shared__ float sgrid[256 * 2];
    for (int i = threadIdx.x; i < n * P; i += blockDim.x) sgrid[i] = grid[i];
    __syncthreads();

    const int lane = threadIdx.x & 31;
    const int64_t groups = K / kGroup;
    const int64_t warp = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (warp >= N * groups) return;
    const int64_t row = warp / groups, gi = warp % groups;

    float v[32];
    load32<T>(W + row * K + gi * kGroup, lane, v);

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

    // scales are stored tile-major: [row / 16][group][row % 16]
    if (lane == 0) scales[((row >> 4) * groups + gi) * 16 + (row & 15)] = __float2half_rn(s * 0.03125f);

    if (P == 2) {
        float best[16];
        int bi[16];
#pragma unroll
        for (int t = 0; t < 16; ++t) { best[t] = INFINITY; bi[t] = 0; }
#pragma unroll 2
        for (int c = 0; c < n; ++c) {
            const float2 gp = *reinterpret_cast<const float2*>(&sgrid[2 * c]);
#pragma unroll
            for (int t = 0; t < 16; ++t) {
                const float dx = v[2 * t] - gp.x, dy = v[2 * t + 1] - gp.y;
                const float d = fmaf(dy, dy, dx * dx);
                if (d < best[t]) { best[t] = d; bi[t] = c; }
            }
        }
        // pair t of chunk c sits at tuple index c*128 + lane*4 + (t&3): 4 consecutive bytes per chunk
        uint8_t* dst = canonical + row * (K / 2) + gi * (kGroup / 2);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t w = (uint32_t)bi[c * 4] | ((uint32_t)bi[c * 4 + 1] << 8) | ((uint32_t)bi[c * 4 + 2] << 16) |
                         ((uint32_t)bi[c * 4 + 3] << 24);
            *reinterpret_cast<uint32_t*>(dst + c * 128 + lane * 4) = w;
        }
    } else {
        float best[32];
        int bi[32];
#pragma unroll
        for (int t = 0; t < 32; ++t) { best[t] = INFINITY; bi[t] = 0; }
#pragma unroll 2
        for (int c = 0; c < n; ++c) {
            const float gp = sgrid[c];
#pragma unroll
            for (int t = 0; t < 32; ++t) {
                const float dx = v[t] - gp;
                const float d = dx * dx;
                if (d < best[t]) { best[t] = d; bi[t] = c; }
            }
        }
        uint8_t* dst = canonical + row * K + gi * kGroup;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t w0 = (uint32_t)bi[c * 8] | ((uint32_t)bi[c * 8 + 1] << 8) | ((uint32_t)bi[c * 8 + 2] << 16) |
                          ((uint32_t)bi[c * 8 + 3] << 24);
            uint32_t w1 = (uint32_t)bi[c * 8 + 4] | ((uint32_t)bi[c * 8 + 5] << 8) | ((uint32_t)bi[c * 8 + 6] << 16) |
                          ((uint32_t)bi[c * 8 + 7] << 24);
            *reinterpret_cast<uint2*>(dst + c * 256 + lane * 8) = make_uint2(w0, w1);
        }
    }
}

// ---- exact pruned search ---------------------------------------------------------------------------------------
// The same nearest-point rule as above, evaluated only on the grid points that can win.  The plane (the line for
// p = 1) is cut into square cells over [-R, R)^p; for a cell, U = min over grid points of the distance to the cell's
// farthest corner bounds the distance of the winner from any point of the cell, so only points whose distance to the
// cell is at most U (+ a slack far above fp32 rounding) can be nearest.  Their indices are listed in ascending order,
// so the strict '<' of the scan keeps the lowest index on ties exactly like the exhaustive scan.  Cells with more
// than kMaxCand candidates, and inputs outside [-R, R)^p, fall back to the exhaustive scan (done by the whole warp for
// one such point at a time: same distances, lowest index on ties).  The table is built once
// by a small kernel (into scratch memory the caller lends: the packed-code output buffer, which is written only after
// the encoder has finished) and copied into shared memory by every persistent encoder block.
constexpr int kCells2 = 64;            // p = 2: 64 x 64 cells of width 1/8 (n = 256: 3 candidates on average, 5 for the
                                       // slowest of a warp's 32 lanes; 32 x 32 cells had 8 and 13)
constexpr int kCells1 = 1024;          // p = 1
constexpr int kMaxCand = 8;            // a cell's list is one 8-byte word
constexpr float kCellR = 4.0f;
constexpr float kCandSlack = 1e-3f;

template <int P>
__global__ void __launch_bounds__(256) build_cells_kernel(const float* __restrict__ grid, int n, uint8_t* __restrict__ table) {
    constexpr int NC = P == 2 ? kCells2 * kCells2 : kCells1;
    __shared__ float sgrid[256 * 2];
    for (int i = threadIdx.x; i < n * P; i += blockDim.x) sgrid[i] = grid[i];
    __syncthreads();
    uint8_t* cand = table;                       // [NC][kMaxCand]
    uint8_t* cnt = table + NC * kMaxCand;        // [NC]
    const float w = 2.0f * kCellR / (P == 2 ? kCells2 : kCells1);
    const int lane = threadIdx.x & 31;
    const int warps = (gridDim.x * blockDim.x) >> 5;
    // one warp per cell; lane l looks at grid points l, l + 32, ... (rounds keep the candidate list in index order)
    for (int cell = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; cell < NC; cell += warps) {
        const float x0 = -kCellR + w * (P == 2 ? (cell % kCells2) : cell), x1 = x0 + w;
        const float y0 = P == 2 ? -kCellR + w * (cell / kCells2) : 0.f, y1 = y0 + w;
        float U = INFINITY;
        for (int c = lane; c < n; c += 32) {
            const float gx = sgrid[P * c], gy = P == 2 ? sgrid[2 * c + 1] : 0.f;
            const float fx = fmaxf(fabsf(gx - x0), fabsf(gx - x1));
            const float fy = P == 2 ? fmaxf(fabsf(gy - y0), fabsf(gy - y1)) : 0.f;
            U = fminf(U, sqrtf(fx * fx + fy * fy));
        }
#pragma unroll
        for (int m = 16; m >= 1; m >>= 1) U = fminf(U, __shfl_xor_sync(0xffffffffu, U, m));
        int k = 0;
        for (int c0 = 0; c0 < n; c0 += 32) {
            const int c = c0 + lane;
            bool in = false;
            if (c < n) {
                const float gx = sgrid[P * c], gy = P == 2 ? sgrid[2 * c + 1] : 0.f;
                const float nx = fmaxf(fmaxf(x0 - gx, gx - x1), 0.f);
                const float ny = P == 2 ? fmaxf(fmaxf(y0 - gy, gy - y1), 0.f) : 0.f;
                in = sqrtf(nx * nx + ny * ny) <= U + kCandSlack;
            }
            const unsigned m = __ballot_sync(0xffffffffu, in);
            const int pos = k + __popc(m & ((1u << lane) - 1u));
            if (in && pos < kMaxCand) cand[cell * kMaxCand + pos] = (uint8_t)c;
            k += __popc(m);
        }
        if (lane == 0) cnt[cell] = k <= kMaxCand ? (uint8_t)k : (uint8_t)255;
    }
}

template <typename T, int P>
__global__ void __launch_bounds__(256) encode_pruned_kernel(const T* __restrict__ W, const float* __restrict__ grid, int n,
                                                            const uint8_t* __restrict__ table,
                                                            uint8_t* __restrict__ canonical, __half* __restrict__ scales,
                                                            int64_t N, int64_t K, uint64_t xi) {
    constexpr int NC = P == 2 ? kCells2 * kCells2 : kCells1;
    __shared__ float sgrid[256 * 2];
    __shared__ __align__(16) uint8_t cand[NC * kMaxCand + NC];
    const uint8_t* cnt = cand + NC * kMaxCand;
    for (int i = threadIdx.x; i < n * P; i += blockDim.x) sgrid[i] = grid[i];
    for (int i = threadIdx.x; i < (NC * kMaxCand + NC) / 16; i += blockDim.x)
        reinterpret_cast<uint4*>(cand)[i] = reinterpret_cast<const uint4*>(table)[i];
    __syncthreads();

    const int lane = threadIdx.x & 31;
    const int64_t groups = K / kGroup;
    const int64_t tasks = N * groups;
    const int64_t warps_total = (int64_t)gridDim.x * (blockDim.x >> 5);
    const float inv_w = (P == 2 ? kCells2 : kCells1) / (2.0f * kCellR);
    for (int64_t task = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); task < tasks; task += warps_total) {
        const int64_t row = task / groups, gi = task % groups;
        float v[32];
        load32<T>(W + row * K + gi * kGroup, lane, v);
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
        if (lane == 0) scales[((row >> 4) * groups + gi) * 16 + (row & 15)] = __float2half_rn(s * 0.03125f);

        int bi[32 / P];
#pragma unroll
        for (int t = 0; t < 32 / P; ++t) {
            const float x = v[P * t], y = P == 2 ? v[2 * t + 1] : 0.f;
            // cell coordinates by rounding down; negative, huge or NaN inputs fail the unsigned comparison
            const int ix = __float2int_rd((x + kCellR) * inv_w), iy = P == 2 ? __float2int_rd((y + kCellR) * inv_w) : 0;
            const bool inside = (unsigned)ix < (unsigned)(P == 2 ? kCells2 : kCells1) && (P == 1 || (unsigned)iy < (unsigned)kCells2);
            const int cell = inside ? (P == 2 ? iy * kCells2 + ix : ix) : 0;
            const int k = inside ? cnt[cell] : 255;
            float best = INFINITY;
            int b = 0;
            // lanes whose point has no candidate list (a crowded outer cell, or outside the table): the warp scans the
            // whole grid for them together, one such lane at a time - left to the lane itself the scan would hold up
            // the other 31 for n iterations whenever any lane needs it
            unsigned full_scan = __ballot_sync(0xffffffffu, k == 255);
            if (k != 255) {
                const uint2 l2 = *reinterpret_cast<const uint2*>(&cand[cell * kMaxCand]);     // the whole list
                for (int i = 0; i < k; ++i) {
                    const int c = (int)(__byte_perm(l2.x, l2.y, (uint32_t)i) & 0xffu);   // byte i of the list
                    const float dx = x - sgrid[P * c], dy = P == 2 ? y - sgrid[2 * c + 1] : 0.f;
                    const float d = P == 2 ? fmaf(dy, dy, dx * dx) : dx * dx;
                    if (d < best) { best = d; b = c; }
                }
            }
            __syncwarp();
            while (full_scan) {
                const int src = __ffs(full_scan) - 1;
                full_scan &= full_scan - 1;
                const float px = __shfl_sync(0xffffffffu, x, src), py = __shfl_sync(0xffffffffu, y, src);
                float bd = INFINITY;
                int bc = 0x7fffffff;
                for (int c = lane; c < n; c += 32) {           // ascending within the lane: '<' keeps its lowest index
                    const float dx = px - sgrid[P * c], dy = P == 2 ? py - sgrid[2 * c + 1] : 0.f;
                    const float d = P == 2 ? fmaf(dy, dy, dx * dx) : dx * dx;
                    if (d < bd) { bd = d; bc = c; }
                }
#pragma unroll
                for (int m = 16; m >= 1; m >>= 1) {             // across lanes: smaller distance, then lower index
                    const float od = __shfl_xor_sync(0xffffffffu, bd, m);
                    const int oc = __shfl_xor_sync(0xffffffffu, bc, m);
                    if (od < bd || (od == bd && oc < bc)) { bd = od; bc = oc; }
                }
                if (lane == src) b = bc;
            }
            bi[t] = b;
        }
        if (P == 2) {
            uint8_t* dst = canonical + row * (K / 2) + gi * (kGroup / 2);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t w = (uint32_t)bi[c * 4] | ((uint32_t)bi[c * 4 + 1] << 8) | ((uint32_t)bi[c * 4 + 2] << 16) |
                             ((uint32_t)bi[c * 4 + 3] << 24);
                *reinterpret_cast<uint32_t*>(dst + c * 128 + lane * 4) = w;
            }
        } else {
            uint8_t* dst = canonical + row * K + gi * kGroup;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t w0 = (uint32_t)bi[c * 8] | ((uint32_t)bi[c * 8 + 1] << 8) | ((uint32_t)bi[c * 8 + 2] << 16) |
                              ((uint32_t)bi[c * 8 + 3] << 24);
                uint32_t w1 = (uint32_t)bi[c * 8 + 4] | ((uint32_t)bi[c * 8 + 5] << 8) | ((uint32_t)bi[c * 8 + 6] << 16) |
                              ((uint32_t)bi[c * 8 + 7] << 24);
                *reinterpret_cast<uint2*>(dst + c * 256 + lane * 8) = make_uint2(w0, w1);
            }
        }
    }
}

// ---- packed layout -----------------------------------------------------------
// The packed stream is a sequence of blocks, block (rt, kb) covering rows
// [16 rt, 16 rt + 16) and inputs [64 kb, 64 kb + 64), stored at block index
// rt * (K/64) + kb.  Inside a block, lane L of the consuming warp owns a
// contiguous run of bytes holding exactly the table indices of the A-fragment
// registers it feeds to four m16n8k16 tensor-core steps: step m (inputs
// 16m..16m+15 of the block), register a in 0..3 is the fp16 pair
//   row   = 16 rt + (L>>2) + 8 (a&1)
//   pairs = inputs 64 kb + 16 m + 2 (L&3) + 8 (a>>1) + {0, 1}.
// "Slot" s = 4m + a, 16 slots per lane.
//   byte-LUT format: 16 bytes per lane, byte s = table index of slot s; a block is
//                    512 contiguous bytes, lane L at byte offset 16 L.
//   six-bit format : three 32-bit words per lane and block.  Words 0 and 1 hold the
//                    low nibbles: slot 4m+a sits in word m>>1 at bit 8a + 4(m&1).
//                    Word 2 holds the high bit-pairs: slot 4m+a at bit 8a + 2m.
//                    (The consumer rebuilds four byte-aligned indices with one shift
//                    and one three-input logic operation each, see linear_mma.cu.)
//   nibble format  : (n = 16) two 32-bit words per lane and block, 256 bytes per block, lane L at
//                    byte offset 8 L.  Byte 2m + h of the lane holds the slots 4m + 2h (low
//                    nibble) and 4m + 2h + 1 (high nibble): the two registers of one row pair.
//   8-bit format   : (p = 1, n = 256) one byte per input: slot 4m + a is the halfword a & 1 of the lane's
//                    word 2m + (a >> 1) (low byte = first input of the pair); a block is 1024 bytes, two
//                    512-byte halves holding words 0..3 and 4..7 of every lane (16 bytes per lane each).
//                    Two neighbouring blocks (2j, 2j+1 along K) form a 768-byte
//                    super-block of three 256-byte planes; plane w stores word w of
//                    lane L, block half h at 32-bit index 2L + h, so a warp reads
//                    each plane with one coalesced 64-bit load per lane.
__device__ __forceinline__ void slot_coords(int64_t rt, int64_t kb, int L, int s, int64_t& row, int64_t& pair) {
    const int m = s >> 2, a = s & 3;
    row = rt * 16 + (L >> 2) + 8 * (a & 1);
    pair = kb * 32 + m * 8 + (L & 3) + 4 * (a >> 1);   // index of the 2-input pair along K
}

// table index of a pair of inputs (2 consecutive k) from the canonical codes
template <int P>
__device__ __forceinline__ uint32_t pair_index(const uint8_t* __restrict__ canonical, int64_t K, int64_t row,
                                               int64_t pair, int bits) {
    if (P == 2) return canonical[row * (K / 2) + pair];
    const uint8_t* q = canonical + row * K + 2 * pair;       // two scalar codes of `bits` bits each
    const uint32_t mask = (1u << bits) - 1u;
    return (uint32_t)(q[0] & mask) | ((uint32_t)(q[1] & mask) << bits);
}

__device__ __forceinline__ void six_bit_store(uint32_t (&w)[3], int s, uint32_t code) {
    const int m = s >> 2, a = s & 3;
    w[m >> 1] |= (code & 15u) << (8 * a + 4 * (m & 1));
    w[2] |= ((code >> 4) & 3u) << (8 * a + 2 * m);
}
__device__ __forceinline__ uint32_t six_bit_load(const uint32_t (&w)[3], int s) {
    const int m = s >> 2, a = s & 3;
    const uint32_t lo = (w[m >> 1] >> (8 * a + 4 * (m & 1))) & 15u;
    const uint32_t hi = (w[2] >> (8 * a + 2 * m)) & 3u;
    return lo | (hi << 4);
}
// 32-bit index of word w of (block kb, lane L) in the six-bit stream
__device__ __forceinline__ int64_t six_bit_word(int64_t rt, int64_t kb, int64_t kblocks, int L, int w) {
    return ((rt * (kblocks >> 1) + (kb >> 1)) * 3 + w) * 64 + 2 * L + (kb & 1);
}

template <int P, int FMT>
__global__ void __launch_bounds__(256) pack_kernel(const uint8_t* __restrict__ canonical, uint32_t* __restrict__ packed,
                                                   int64_t N, int64_t K, int bits) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t kblocks = K / kBlockK;
    const int64_t total = (N / 16) * kblocks * 32;
    if (t >= total) return;
    const int L = (int)(t & 31);
    const int64_t blk = t >> 5, rt = blk / kblocks, kb = blk % kblocks;
    constexpr bool SIX = FMT == 1, NIB = FMT == 2, B8 = FMT == 3;
    if (B8) {
        uint32_t w[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
        for (int s = 0; s < 16; ++s) {
            int64_t row, pair;
            slot_coords(rt, kb, L, s, row, pair);
            const uint8_t* q = canonical + row * K + 2 * pair;
            w[2 * (s >> 2) + ((s & 3) >> 1)] |= ((uint32_t)q[0] | ((uint32_t)q[1] << 8)) << (16 * (s & 1));
        }
        uint4* out = reinterpret_cast<uint4*>(packed) + blk * 64;      // 1024-byte block = 64 uint4
        out[L] = make_uint4(w[0], w[1], w[2], w[3]);
        out[32 + L] = make_uint4(w[4], w[5], w[6], w[7]);
    } else if (SIX) {
        uint32_t w[3] = {0u, 0u, 0u};
        for (int s = 0; s < 16; ++s) {
            int64_t row, pair;
            slot_coords(rt, kb, L, s, row, pair);
            six_bit_store(w, s, pair_index<P>(canonical, K, row, pair, bits) & 63u);
        }
        for (int i = 0; i < 3; ++i) packed[six_bit_word(rt, kb, kblocks, L, i)] = w[i];
    } else if (NIB) {
        uint32_t w[2] = {0u, 0u};
        for (int s = 0; s < 16; ++s) {
            int64_t row, pair;
            slot_coords(rt, kb, L, s, row, pair);
            const int m = s >> 2, a = s & 3, byte = 2 * m + (a >> 1);
            w[byte >> 2] |= (pair_index<P>(canonical, K, row, pair, bits) & 15u) << (8 * (byte & 3) + 4 * (a & 1));
        }
        reinterpret_cast<uint2*>(packed)[t] = make_uint2(w[0], w[1]);
    } else {
        uint32_t w[4] = {0u, 0u, 0u, 0u};
        for (int s = 0; s < 16; ++s) {
            int64_t row, pair;
            slot_coords(rt, kb, L, s, row, pair);
            w[s >> 2] |= pair_index<P>(canonical, K, row, pair, bits) << (8 * (s & 3));
        }
        reinterpret_cast<uint4*>(packed)[t] = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

template <int P, int FMT>
__global__ void __launch_bounds__(256) unpack_kernel(const uint32_t* __restrict__ packed, uint8_t* __restrict__ canonical,
                                                     int64_t N, int64_t K, int bits) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t kblocks = K / kBlockK;
    const int64_t total = (N / 16) * kblocks * 32;
    if (t >= total) return;
    const int L = (int)(t & 31);
    const int64_t blk = t >> 5, rt = blk / kblocks, kb = blk % kblocks;
    constexpr bool SIX = FMT == 1, NIB = FMT == 2, B8 = FMT == 3;
    if (B8) {
        const uint4* in = reinterpret_cast<const uint4*>(packed) + blk * 64;
        const uint4 q0 = in[L], q1 = in[32 + L];
        const uint32_t w[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
        for (int s = 0; s < 16; ++s) {
            int64_t row, pair;
            slot_coords(rt, kb, L, s, row, pair);
            const uint32_t hw = (w[2 * (s >> 2) + ((s & 3) >> 1)] >> (16 * (s & 1))) & 0xffffu;
            canonical[row * K + 2 * pair] = (uint8_t)(hw & 255u);
            canonical[row * K + 2 * pair + 1] = (uint8_t)(hw >> 8);
        }
        return;
    }
    uint32_t w6[3] = {0u, 0u, 0u};
    uint32_t w8[4] = {0u, 0u, 0u, 0u};
    if (SIX) {
        for (int i = 0; i < 3; ++i) w6[i] = packed[six_bit_word(rt, kb, kblocks, L, i)];
    } else if (NIB) {
        uint2 q = reinterpret_cast<const uint2*>(packed)[t];
        w8[0] = q.x; w8[1] = q.y;
    } else {
        uint4 q = reinterpret_cast<const uint4*>(packed)[t];
        w8[0] = q.x; w8[1] = q.y; w8[2] = q.z; w8[3] = q.w;
    }
    for (int s = 0; s < 16; ++s) {
        int64_t row, pair;
        slot_coords(rt, kb, L, s, row, pair);
        const int nbyte = 2 * (s >> 2) + ((s & 3) >> 1);       // nibble format: byte of the lane holding slot s
        const uint32_t idx = SIX ? six_bit_load(w6, s)
                           : NIB ? ((w8[nbyte >> 2] >> (8 * (nbyte & 3) + 4 * (s & 1))) & 15u)
                                 : ((w8[s >> 2] >> (8 * (s & 3))) & 255u);
        if (P == 2) {
            canonical[row * (K / 2) + pair] = (uint8_t)idx;
        } else {
            canonical[row * K + 2 * pair] = (uint8_t)(idx & ((1u << bits) - 1u));
            canonical[row * K + 2 * pair + 1] = (uint8_t)((idx >> bits) & ((1u << bits) - 1u));
        }
    }
}

}  // namespace

int launch_encode(const higgs_desc& d, const void* W, int w_dtype, const float* grid, uint8_t* canonical, void* scales,
                  void* scratch, size_t scratch_bytes, cudaStream_t st) {
    const int64_t warps = d.N * (d.K / kGroup);
    if (warps == 0) return HIGGS_OK;
    const unsigned blocks = (unsigned)((warps + 3) / 4);
    __half* sc = static_cast<__half*>(scales);
    // Large grids on large layers: the exact pruned search (persistent blocks that build their candidate table once);
    // otherwise the exhaustive scan, whose cost is small there.
    constexpr size_t kTableBytes = (size_t)(kCells1 > kCells2 * kCells2 ? kCells1 : kCells2 * kCells2) * (kMaxCand + 1);
    const bool pruned = d.n >= 64 && warps >= 2048 && scratch && scratch_bytes >= kTableBytes &&
                        (reinterpret_cast<uintptr_t>(scratch) % 16) == 0;
    const unsigned pblocks = 592;          // 4 blocks of 8 warps per SM on a 148-SM part; any count is correct
    uint8_t* table = static_cast<uint8_t*>(scratch);
    if (pruned) {
        if (d.p == 2) build_cells_kernel<2><<<128, 256, 0, st>>>(grid, d.n, table);      // one warp per cell
        else build_cells_kernel<1><<<128, 256, 0, st>>>(grid, d.n, table);
    }
#define HIGGS_ENC(T, P) \
    if (pruned) encode_pruned_kernel<T, P><<<pblocks, 256, 0, st>>>(static_cast<const T*>(W), grid, d.n, table, canonical, sc, d.N, d.K, d.rht_seed); \
    else encode_kernel<T, P><<<blocks, 128, 0, st>>>(static_cast<const T*>(W), grid, d.n, canonical, sc, d.N, d.K, d.rht_seed)
    if (w_dtype == HIGGS_F32 && d.p == 2) { HIGGS_ENC(float, 2); }
    else if (w_dtype == HIGGS_F32 && d.p == 1) { HIGGS_ENC(float, 1); }
    else if (w_dtype == HIGGS_BF16 && d.p == 2) { HIGGS_ENC(__nv_bfloat16, 2); }
    else if (w_dtype == HIGGS_BF16 && d.p == 1) { HIGGS_ENC(__nv_bfloat16, 1); }
    else return HIGGS_ERR_UNSUPPORTED;
#undef HIGGS_ENC
    return cuda_status(cudaGetLastError());
}

int launch_pack(const higgs_desc& d, const uint8_t* canonical, void* packed, cudaStream_t st) {
    const int64_t total = (d.N / 16) * (d.K / kBlockK) * 32;
    if (total == 0) return HIGGS_OK;
    const unsigned blocks = (unsigned)((total + 255) / 256);
    uint32_t* out = static_cast<uint32_t*>(packed);
    const Format f = format_of(d.p, d.n);
    const int bits = code_bits(d.n);
    if (f == Format::kByteLut && d.p == 2) pack_kernel<2, 0><<<blocks, 256, 0, st>>>(canonical, out, d.N, d.K, bits);
    else if (f == Format::kByteLut && d.p == 1) pack_kernel<1, 0><<<blocks, 256, 0, st>>>(canonical, out, d.N, d.K, bits);
    else if (f == Format::kSixBit && d.p == 2) pack_kernel<2, 1><<<blocks, 256, 0, st>>>(canonical, out, d.N, d.K, bits);
    else if (f == Format::kSixBit) pack_kernel<1, 1><<<blocks, 256, 0, st>>>(canonical, out, d.N, d.K, bits);
    else if (f == Format::kNibble && d.p == 2) pack_kernel<2, 2><<<blocks, 256, 0, st>>>(canonical, out, d.N, d.K, bits);
    else if (f == Format::kNibble) pack_kernel<1, 2><<<blocks, 256, 0, st>>>(canonical, out, d.N, d.K, bits);
    else if (f == Format::kByte8) pack_kernel<1, 3><<<blocks, 256, 0, st>>>(canonical, out, d.N, d.K, bits);
    else return HIGGS_ERR_UNSUPPORTED;
    return cuda_status(cudaGetLastError());
}

int launch_unpack(const higgs_desc& d, const void* packed, uint8_t* canonical, cudaStream_t st) {
    const int64_t total = (d.N / 16) * (d.K / kBlockK) * 32;
    if (total == 0) return HIGGS_OK;
    const unsigned blocks = (unsigned)((total + 255) / 256);
    const uint32_t* in = static_cast<const uint32_t*>(packed);
    const Format f = format_of(d.p, d.n);
    const int bits = code_bits(d.n);
    if (f == Format::kByteLut && d.p == 2) unpack_kernel<2, 0><<<blocks, 256, 0, st>>>(in, canonical, d.N, d.K, bits);
    else if (f == Format::kByteLut && d.p == 1) unpack_kernel<1, 0><<<blocks, 256, 0, st>>>(in, canonical, d.N, d.K, bits);
    else if (f == Format::kSixBit && d.p == 2) unpack_kernel<2, 1><<<blocks, 256, 0, st>>>(in, canonical, d.N, d.K, bits);
    else if (f == Format::kSixBit) unpack_kernel<1, 1><<<blocks, 256, 0, st>>>(in, canonical, d.N, d.K, bits);
    else if (f == Format::kNibble && d.p == 2) unpack_kernel<2, 2><<<blocks, 256, 0, st>>>(in, canonical, d.N, d.K, bits);
    else if (f == Format::kNibble) unpack_kernel<1, 2><<<blocks, 256, 0, st>>>(in, canonical, d.N, d.K, bits);
    else if (f == Format::kByte8) unpack_kernel<1, 3><<<blocks, 256, 0, st>>>(in, canonical, d.N, d.K, bits);
    else return HIGGS_ERR_UNSUPPORTED;
    return cuda_status(cudaGetLastError());
}

}  // namespace higgs
