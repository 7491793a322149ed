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

// The packed words of one (64-input block, lane) position, assembled from a tile of canonical codes in shared memory
// (16 rows of the row tile, RS bytes apart; kbl = the 64-input block inside the tile's 1024 inputs) and stored.
// fmt: 0 byte, 1 six-bit, 2 nibble, 3 8-bit (uniform over the block).
template <int P>
__device__ __forceinline__ void pack_item(const uint8_t* tile, int RS, int fmt, int bits, int kbl, int L, int64_t rt,
                                          int64_t kb, int64_t kblocks, uint32_t* __restrict__ packed) {
    const int64_t blk = rt * kblocks + kb, t = blk * 32 + L;
    const uint32_t mask = (1u << bits) - 1u;
    // table index of slot s = 4m + a of this lane (two consecutive inputs): row (L>>2) + 8(a&1) of the tile,
    // pair kbl*32 + m*8 + (L&3) + 4(a>>1)
    auto index_of = [&](int s) -> uint32_t {
        const int m = s >> 2, a = s & 3;
        const int row = (L >> 2) + 8 * (a & 1), pair = kbl * 32 + m * 8 + (L & 3) + 4 * (a >> 1);
        if (P == 2) return tile[row * RS + pair];
        const uint8_t* q = tile + row * RS + 2 * pair;       // two scalar codes of `bits` bits each
        return (uint32_t)(q[0] & mask) | ((uint32_t)(q[1] & mask) << bits);
    };
    if (P == 1 && fmt == 3) {
        uint32_t w[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
#pragma unroll
        for (int s = 0; s < 16; ++s) w[2 * (s >> 2) + ((s & 3) >> 1)] |= index_of(s) << (16 * (s & 1));
        uint4* out = reinterpret_cast<uint4*>(packed) + blk * 64;      // 1024-byte block = 64 uint4
        out[L] = make_uint4(w[0], w[1], w[2], w[3]);
        out[32 + L] = make_uint4(w[4], w[5], w[6], w[7]);
    } else if (fmt == 1) {
        uint32_t w[3] = {0u, 0u, 0u};
#pragma unroll
        for (int s = 0; s < 16; ++s) six_bit_store(w, s, index_of(s) & 63u);
#pragma unroll
        for (int i = 0; i < 3; ++i) packed[six_bit_word(rt, kb, kblocks, L, i)] = w[i];
    } else if (fmt == 2) {
        uint32_t w[2] = {0u, 0u};
#pragma unroll
        for (int s = 0; s < 16; ++s) {
            const int m = s >> 2, a = s & 3, byte = 2 * m + (a >> 1);
            w[byte >> 2] |= (index_of(s) & 15u) << (8 * (byte & 3) + 4 * (a & 1));
        }
        reinterpret_cast<uint2*>(packed)[t] = make_uint2(w[0], w[1]);
    } else {
        uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int s = 0; s < 16; ++s) w[s >> 2] |= index_of(s) << (8 * (s & 3));
        reinterpret_cast<uint4*>(packed)[t] = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

__host__ __device__ constexpr int kTileRowBytes(int P) { return (P == 2 ? 512 : 1024) + 16; }   // rows 16 bytes apart in bank position

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
// p = 1) is cut into square cells; cell i of an axis covers the values whose scaled coordinate x * cells / 2R + cells / 2
// rounds to i (found with one fused multiply-add onto 2^23: the integer is then the low bits of the float).  A cell's
// candidate list is built in two steps.  (1) U = min over grid points of the distance to the cell's farthest corner
// bounds the winner's distance from any point of the cell, so only points whose distance to the cell is at most U (+ a
// slack far above fp32 rounding) can be nearest.  (2) Of those, c is dropped if another candidate c' is nearer at all
// corners of the cell by a margin: |z - c|^2 - |z - c'|^2 is affine in z, so its minimum over the cell is at a corner,
// and c wins nowhere in the cell.  The surviving indices (at most four - two for p = 1 -, else the cell is marked) are stored in
// ascending order, the last one repeated up to four: the encoder evaluates all four without a branch, and its strict
// '<' keeps the lowest index on ties exactly like the exhaustive scan (a repeated candidate never replaces itself).
// Marked cells and inputs outside the table take the exhaustive scan, done by the whole warp for one such point at a
// time, after the warp's other points: same distances, lowest index on ties.  The table is built once per call by a
// small kernel (into scratch memory the caller lends: the packed-code output buffer, which is written only after the
// encoder has finished) and copied into shared memory by every persistent encoder block.
constexpr int kCells2 = 128;           // p = 2: 128 x 128 cells of width 1/16 (n = 256: 1.6 candidates on average, at most 4)
constexpr int kCells1 = 1024;          // p = 1: width 1/128, at most 2 candidates
constexpr int kMaxCand = 4;            // a cell's list is one 32-bit word
constexpr int kPrefilter = 32;         // candidates that step (1) may leave for step (2)
constexpr uint32_t kCellScan = 1u;     // bytes (1, 0, 0, 0) are not an ascending list: the cell needs the exhaustive scan
constexpr float kCellR = 4.0f;
constexpr float kCandSlack = 1e-3f;
constexpr float kDominance = 1e-3f;    // margin of step (2) on squared distances (fp32 rounding there is below 1e-5)

template <int P>
__global__ void __launch_bounds__(256) build_cells_kernel(const float* __restrict__ grid, int n, uint32_t* __restrict__ table) {
    constexpr int NC = P == 2 ? kCells2 * kCells2 : kCells1;
    constexpr int CELLS = P == 2 ? kCells2 : kCells1;
    __shared__ float sgrid[256 * 2];
    __shared__ int slist[8][kPrefilter];
    for (int i = threadIdx.x; i < n * P; i += blockDim.x) sgrid[i] = grid[i];
    __syncthreads();
    const float w = 2.0f * kCellR / CELLS;
    const int lane = threadIdx.x & 31, wi = threadIdx.x >> 5;
    const int warps = (gridDim.x * blockDim.x) >> 5;
    // one warp per cell; lane l looks at grid points l, l + 32, ... (rounds keep the candidate list in index order)
    for (int cell = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; cell < NC; cell += warps) {
        const int cx = P == 2 ? cell % kCells2 : cell, cy = P == 2 ? cell / kCells2 : 0;
        const float x0 = w * ((float)cx - 0.5f - 0.5f * CELLS), x1 = x0 + w;
        const float y0 = P == 2 ? w * ((float)cy - 0.5f - 0.5f * CELLS) : 0.f, y1 = y0 + w;
        float U2 = INFINITY;
        for (int c = lane; c < n; c += 32) {
            const float gx = sgrid[P * c], gy = P == 2 ? sgrid[2 * c + 1] : 0.f;
            const float fx = fmaxf(fabsf(gx - x0), fabsf(gx - x1));
            const float fy = P == 2 ? fmaxf(fabsf(gy - y0), fabsf(gy - y1)) : 0.f;
            U2 = fminf(U2, fx * fx + fy * fy);
        }
#pragma unroll
        for (int m = 16; m >= 1; m >>= 1) U2 = fminf(U2, __shfl_xor_sync(0xffffffffu, U2, m));
        const float reach = sqrtf(U2) + kCandSlack, reach2 = reach * reach;
        int k = 0;
        for (int c0 = 0; c0 < n; c0 += 32) {
            const int c = c0 + lane;
            bool in = false;
            if (c < n) {
                const float gx = sgrid[P * c], gy = P == 2 ? sgrid[2 * c + 1] : 0.f;
                const float nx = fmaxf(fmaxf(x0 - gx, gx - x1), 0.f);
                const float ny = P == 2 ? fmaxf(fmaxf(y0 - gy, gy - y1), 0.f) : 0.f;
                in = nx * nx + ny * ny <= reach2;
            }
            const unsigned m = __ballot_sync(0xffffffffu, in);
            const int pos = k + __popc(m & ((1u << lane) - 1u));
            if (in && pos < kPrefilter) slist[wi][pos] = c;
            k += __popc(m);
        }
        __syncwarp();
        uint32_t word = kCellScan;
        if (k <= kPrefilter) {
            // step (2): lane i judges candidate i against every candidate j
            const bool have = lane < k;
            const int mine = have ? slist[wi][lane] : 0;
            const float mx = sgrid[P * mine], my = P == 2 ? sgrid[2 * mine + 1] : 0.f;
            const float qx[2] = {x0, x1}, qy[2] = {y0, y1};
            float dm[4];
#pragma unroll
            for (int q = 0; q < (P == 2 ? 4 : 2); ++q) {
                const float dx = qx[q & 1] - mx, dy = P == 2 ? qy[q >> 1] - my : 0.f;
                dm[q] = dx * dx + dy * dy;
            }
            bool dominated = false;
            for (int j = 0; j < k; ++j) {
                const int cj = slist[wi][j];
                const float gx = sgrid[P * cj], gy = P == 2 ? sgrid[2 * cj + 1] : 0.f;
                bool all = true;
#pragma unroll
                for (int q = 0; q < (P == 2 ? 4 : 2); ++q) {
                    const float dx = qx[q & 1] - gx, dy = P == 2 ? qy[q >> 1] - gy : 0.f;
                    all = all && (dx * dx + dy * dy + kDominance < dm[q]);
                }
                dominated = dominated || all;
            }
            const unsigned kept = __ballot_sync(0xffffffffu, have && !dominated);
            const int cnt = __popc(kept);
            if (cnt >= 1 && cnt <= (P == 2 ? kMaxCand : 2)) {      // the encoder evaluates four candidates for p = 2, two for p = 1
                // the kept lane of rank r supplies byte r; the last one also fills the bytes above it
                const int r = __popc(kept & ((1u << lane) - 1u));
                const bool is_kept = (kept >> lane) & 1u;
                const uint32_t part = !is_kept ? 0u : (r == cnt - 1 ? (uint32_t)mine * (0x01010101u << (8 * r)) : (uint32_t)mine << (8 * r));
                word = __reduce_or_sync(0xffffffffu, part);
            }
        }
        if (lane == 0) table[cell] = word;
        __syncwarp();
    }
}

// status of the encoder's bounded waits (HIGGS_ERR_TIMEOUT if one ran out), read by higgs_device_status
__device__ int g_encode_status = 0;
constexpr uint32_t kEncodeWaitLimit = 1u << 22;

__device__ __forceinline__ uint32_t enc_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void enc_mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void enc_mbar_arrive(uint32_t bar) {
    asm volatile("{\n\t.reg .b64 t;\n\tmbarrier.arrive.shared::cta.b64 t, [%0];\n\t}" ::"r"(bar) : "memory");
}
// waits for the phase of the given parity, at most kEncodeWaitLimit polls; a wait that runs out is recorded and the
// caller carries on (wrong codes for that launch, which the status word reports, rather than a hung device)
__device__ __forceinline__ void enc_mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t it = 0; it < kEncodeWaitLimit; ++it) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (done) return;
    }
    atomicExch(&g_encode_status, (int)HIGGS_ERR_TIMEOUT);
}

// the exhaustive scan of one point by the whole warp (lowest index among equal distances); point c is the first
// eight (four for p = 1) bytes of row c of the replicated grid
template <int P>
__device__ __noinline__ int warp_scan(const uint8_t* rep, int n, float px, float py, int lane) {
    float bd = INFINITY;
    int bc = 0x7fffffff;
    for (int c = lane; c < n; c += 32) {           // ascending within the lane: '<' keeps its lowest index
        const float* g = reinterpret_cast<const float*>(rep + c * 128);
        const float dx = px - g[0], dy = P == 2 ? py - g[1] : 0.f;
        const float d = P == 2 ? fmaf(dy, dy, dx * dx) : dx * dx;
        if (d < bd) { bd = d; bc = c; }
    }
#pragma unroll
    for (int m = 16; m >= 1; m >>= 1) {             // across lanes: smaller distance, then lower index
        const float od = __shfl_xor_sync(0xffffffffu, bd, m);
        const int oc = __shfl_xor_sync(0xffffffffu, bc, m);
        if (od < bd || (od == bd && oc < bc)) { bd = od; bc = oc; }
    }
    return bc == 0x7fffffff ? 0 : bc;               // no distance compared below infinity (a NaN input): index 0, as the scan
}

// Persistent blocks of 16 warps; a block takes one row tile (16 rows) x one group per turn, warp w the tile's row w.
// Shared memory: the cell table; the grid with every point repeated across a 128-byte row (16 copies of an 8-byte
// point for p = 2, 32 copies of a float for p = 1: a lane reads "its" copy and the 32 lookups of a warp never meet in
// a bank); two tiles of canonical codes, through which the block emits the packed stream itself (thread t assembles
// the words of 64-input block t / 32, lane t % 32).  The warps of a block are not held in step: a warp puts its row
// into the turn's tile and arrives on an mbarrier, and only a turn later - after its next search - waits for that
// phase and packs the finished tile, so a warp may run up to one turn ahead of the slowest (a block-wide barrier per
// turn made all sixteen warps wait for memory together and cost 20 %).  Writing tile t % 2 in turn t is safe: it was
// last read when every warp packed tile t - 2, before its arrival of turn t - 1, which this warp has waited for.
// canonical and packed may each be null (not both).
template <typename T, int P>
__global__ void __launch_bounds__(512, 2) encode_pruned_kernel(const T* __restrict__ W, const float* __restrict__ grid, int n,
                                                               const uint32_t* __restrict__ table,
                                                               uint8_t* __restrict__ canonical, uint32_t* __restrict__ packed,
                                                               int fmt, int bits, __half* __restrict__ scales,
                                                               int64_t N, int64_t K, uint64_t xi) {
    constexpr int NC = P == 2 ? kCells2 * kCells2 : kCells1;
    constexpr int CELLS = P == 2 ? kCells2 : kCells1;
    constexpr int RS = kTileRowBytes(P);
    extern __shared__ __align__(128) uint8_t enc_smem[];
    uint32_t* cells = reinterpret_cast<uint32_t*>(enc_smem);
    uint8_t* rep = enc_smem + (size_t)NC * 4;
    uint8_t* tiles_base = rep + (size_t)n * 128;
    const uint32_t bar = enc_smem_u32(tiles_base + 2 * 16 * RS);      // mbarrier: one arrival per warp and turn
    if (threadIdx.x == 0) enc_mbar_init(bar, 16);
    for (int i = threadIdx.x; i < NC / 4; i += blockDim.x)
        reinterpret_cast<uint4*>(cells)[i] = reinterpret_cast<const uint4*>(table)[i];
    for (int i = threadIdx.x; i < n * 32; i += blockDim.x)
        reinterpret_cast<float*>(rep)[i] = grid[P == 2 ? 2 * (i >> 5) + (i & 1) : (i >> 5)];
    __syncthreads();

    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const uint8_t* rep_lane = rep + (P == 2 ? (lane & 15) * 8 : lane * 4);
    const int64_t groups = K / kGroup, kblocks = K / kBlockK;
    const int64_t turns = (N / 16) * groups;
    const float inv_w = CELLS / (2.0f * kCellR);
    const float magic = 8388608.0f + 0.5f * CELLS;
    // (row tile, group) of the block's turn, advanced by the grid's stride without a division per turn
    int64_t rt = (int64_t)blockIdx.x / groups, gi = (int64_t)blockIdx.x % groups;
    const int64_t step_tiles = (int64_t)gridDim.x / groups, step_groups = (int64_t)gridDim.x % groups;
    int parity = 0;                  // tile of this turn
    int64_t prev_rt = -1, prev_gi = 0;
    for (int64_t turn = blockIdx.x; turn < turns; turn += gridDim.x, rt += step_tiles, gi += step_groups, parity ^= 1) {
        if (gi >= groups) { gi -= groups; ++rt; }
        const int64_t row = rt * 16 + wib;
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
        if (lane == 0) scales[(rt * groups + gi) * 16 + wib] = __float2half_rn(s * 0.03125f);

        uint32_t out[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};      // the lane's codes, one byte each, in storage order
        uint32_t slow = 0u;                                       // bit t: tuple t needs the exhaustive scan
#pragma unroll
        for (int t = 0; t < 32 / P; ++t) {
            const float x = v[P * t], y = P == 2 ? v[2 * t + 1] : 0.f;
            // the float 2^23 + i carries i in its low bits; anything else (outside the table, NaN) leaves other bits set
            const uint32_t ix = __float_as_uint(fmaf(x, inv_w, magic)) ^ 0x4B000000u;
            const uint32_t iy = P == 2 ? __float_as_uint(fmaf(y, inv_w, magic)) ^ 0x4B000000u : 0u;
            const bool inside = (ix | iy) < (uint32_t)CELLS;
            uint32_t list = kCellScan;
            if (inside) list = cells[P == 2 ? iy * kCells2 + ix : ix];
            if (list == kCellScan) { slow |= 1u << t; list = 0u; }
            float best;
            uint32_t b;
#pragma unroll
            for (int i = 0; i < (P == 2 ? kMaxCand : 2); ++i) {
                const uint32_t c = __byte_perm(list, 0u, 0x4440u + i);
                float d;
                if (P == 2) {
                    const float2 g = *reinterpret_cast<const float2*>(rep_lane + c * 128u);
                    const float dx = x - g.x, dy = y - g.y;
                    d = fmaf(dy, dy, dx * dx);
                } else {
                    const float dx = x - *reinterpret_cast<const float*>(rep_lane + c * 128u);
                    d = dx * dx;
                }
                if (i == 0 || d < best) { best = d; b = c; }
            }
            out[t >> 2] |= b << (8 * (t & 3));
        }
        if (__any_sync(0xffffffffu, slow != 0u)) {
#pragma unroll
            for (int t = 0; t < 32 / P; ++t) {
                unsigned m = __ballot_sync(0xffffffffu, (slow >> t) & 1u);
                while (m) {
                    const int src = __ffs(m) - 1;
                    m &= m - 1;
                    const float px = __shfl_sync(0xffffffffu, v[P * t], src);
                    const float py = P == 2 ? __shfl_sync(0xffffffffu, v[2 * t + 1], src) : 0.f;
                    const int bc = warp_scan<P>(rep, n, px, py, lane);
                    if (lane == src) out[t >> 2] = (out[t >> 2] & ~(0xffu << (8 * (t & 3)))) | ((uint32_t)bc << (8 * (t & 3)));
                }
            }
        }
        // tuple t of chunk c sits at tuple index c*128 + lane*4 + (t&3) (p = 2: four consecutive bytes per chunk);
        // value t of chunk c at c*256 + lane*8 + t (p = 1: eight)
        if (canonical) {
            if (P == 2) {
                uint8_t* dst = canonical + row * (K / 2) + gi * (kGroup / 2);
#pragma unroll
                for (int c = 0; c < 4; ++c) *reinterpret_cast<uint32_t*>(dst + c * 128 + lane * 4) = out[c];
            } else {
                uint8_t* dst = canonical + row * K + gi * kGroup;
#pragma unroll
                for (int c = 0; c < 4; ++c) *reinterpret_cast<uint2*>(dst + c * 256 + lane * 8) = make_uint2(out[2 * c], out[2 * c + 1]);
            }
        }
        if (packed) {
            if (prev_rt >= 0) {      // the tile of the turn before: complete once all sixteen warps have arrived
                enc_mbar_wait(bar, (uint32_t)(parity ^ 1));
                pack_item<P>(tiles_base + (parity ^ 1) * (16 * RS), RS, fmt, bits, wib, lane, prev_rt, prev_gi * 16 + wib, kblocks, packed);
            }
            uint8_t* mine = tiles_base + parity * (16 * RS) + wib * RS;
            if (P == 2) {
#pragma unroll
                for (int c = 0; c < 4; ++c) *reinterpret_cast<uint32_t*>(mine + c * 128 + lane * 4) = out[c];
            } else {
#pragma unroll
                for (int c = 0; c < 4; ++c) *reinterpret_cast<uint2*>(mine + c * 256 + lane * 8) = make_uint2(out[2 * c], out[2 * c + 1]);
            }
            __syncwarp();
            if (lane == 0) enc_mbar_arrive(bar);
            prev_rt = rt;
            prev_gi = gi;
        }
    }
    if (packed && prev_rt >= 0) {
        enc_mbar_wait(bar, (uint32_t)(parity ^ 1));
        pack_item<P>(tiles_base + (parity ^ 1) * (16 * RS), RS, fmt, bits, wib, lane, prev_rt, prev_gi * 16 + wib, kblocks, packed);
    }
}

// One block packs 16 rows x 1024 inputs: the canonical codes of the tile are staged in shared memory with coalesced
// 16-byte loads (no bank conflicts in the byte gathers, see kTileRowBytes), then every thread assembles the words of
// two (64-input block, lane) positions and stores them coalesced.
template <int P>
__global__ void __launch_bounds__(256) pack_kernel(const uint8_t* __restrict__ canonical, uint32_t* __restrict__ packed,
                                                   int64_t N, int64_t K, int fmt, int bits) {
    constexpr int RS = kTileRowBytes(P), RB = RS - 16;          // RB canonical bytes of one row and 1024 inputs
    __shared__ __align__(16) uint8_t tile[16 * RS];
    const int64_t kblocks = K / kBlockK, ktiles = K / kGroup;
    const int64_t rt = blockIdx.x / ktiles, kt = blockIdx.x % ktiles;
    for (int i = threadIdx.x; i < 16 * (RB / 16); i += 256) {
        const int r = i / (RB / 16), c = i % (RB / 16);
        *reinterpret_cast<uint4*>(tile + r * RS + c * 16) =
            *reinterpret_cast<const uint4*>(canonical + ((rt * 16 + r) * ktiles + kt) * RB + c * 16);
    }
    __syncthreads();
    for (int item = threadIdx.x; item < 512; item += 256)
        pack_item<P>(tile, RS, fmt, bits, item >> 5, item & 31, rt, kt * 16 + (item >> 5), kblocks, packed);
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

int sm_count() {
    static int cached[64] = {0};
    return device_once(cached, [] {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0)
            v = 148;
        return v;
    });
}

}  // namespace

int read_encode_status(int clear) {
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_encode_status, sizeof(int)) != cudaSuccess) return HIGGS_ERR_CUDA;
    if (clear && v != 0) {
        const int zero = 0;
        if (cudaMemcpyToSymbol(g_encode_status, &zero, sizeof(int)) != cudaSuccess) return HIGGS_ERR_CUDA;
    }
    return v;
}

size_t encoder_table_bytes(int p) { return (size_t)(p == 2 ? kCells2 * kCells2 : kCells1) * 4; }

int launch_encoder_table(int p, int n, const float* grid, void* table, cudaStream_t st) {
    if (p == 2) build_cells_kernel<2><<<592, 256, 0, st>>>(grid, n, static_cast<uint32_t*>(table));      // one warp per cell and turn
    else build_cells_kernel<1><<<128, 256, 0, st>>>(grid, n, static_cast<uint32_t*>(table));
    return cuda_status(cudaGetLastError());
}

// table: a prepared cell table, or null; build_space: where to build one (encoder_table_bytes, 16-byte aligned), or
// null.  Large layers with a table take the pruned search, which also emits the packed stream when `packed` is given
// (*packed_done = true); everything else is the exhaustive scan into `canonical`.
int launch_encode(const higgs_desc& d, const void* W, int w_dtype, const float* grid, const void* table, void* build_space,
                  uint8_t* canonical, void* packed, void* scales, bool* packed_done, cudaStream_t st) {
    *packed_done = false;
    const int64_t warps = d.N * (d.K / kGroup);
    if (warps == 0) return HIGGS_OK;
    __half* sc = static_cast<__half*>(scales);
    const bool pruned = warps >= kPrunedMinTasks && (table || build_space) && (canonical || packed);
    if (!pruned) {
        if (!canonical) return HIGGS_ERR_INVALID_ARG;
        const unsigned blocks = (unsigned)((warps + 3) / 4);
#define HIGGS_ENC(T, P) encode_kernel<T, P><<<blocks, 128, 0, st>>>(static_cast<const T*>(W), grid, d.n, canonical, sc, d.N, d.K, d.rht_seed)
        if (w_dtype == HIGGS_F32 && d.p == 2) HIGGS_ENC(float, 2);
        else if (w_dtype == HIGGS_F32 && d.p == 1) HIGGS_ENC(float, 1);
        else if (w_dtype == HIGGS_BF16 && d.p == 2) HIGGS_ENC(__nv_bfloat16, 2);
        else if (w_dtype == HIGGS_BF16 && d.p == 1) HIGGS_ENC(__nv_bfloat16, 1);
        else return HIGGS_ERR_UNSUPPORTED;
#undef HIGGS_ENC
        return cuda_status(cudaGetLastError());
    }
    static int configured[64];
    const int ok = device_once(configured, [] {
        constexpr int kMax = kCells2 * kCells2 * 4 + 256 * 128 + 2 * 16 * kTileRowBytes(1) + 16;
        bool good = true;
        good = good && cudaFuncSetAttribute(encode_pruned_kernel<float, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMax) == cudaSuccess;
        good = good && cudaFuncSetAttribute(encode_pruned_kernel<float, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMax) == cudaSuccess;
        good = good && cudaFuncSetAttribute(encode_pruned_kernel<__nv_bfloat16, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMax) == cudaSuccess;
        good = good && cudaFuncSetAttribute(encode_pruned_kernel<__nv_bfloat16, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMax) == cudaSuccess;
        return good ? 1 : -1;
    });
    if (ok < 0) return HIGGS_ERR_CUDA;
    if (!table) {
        const int rc = launch_encoder_table(d.p, d.n, grid, build_space, st);
        if (rc != HIGGS_OK) return rc;
        table = build_space;
    }
    const uint32_t* tab = static_cast<const uint32_t*>(table);
    uint32_t* pk = static_cast<uint32_t*>(packed);
    const size_t smem = encoder_table_bytes(d.p) + (size_t)d.n * 128 + 2 * 16 * (size_t)kTileRowBytes(d.p) + 16;
    const int64_t turns = (d.N / 16) * (d.K / kGroup);
    const int fmt = (int)format_of(d.p, d.n) - 1, bits = code_bits(d.n);
    // persistent grid: as many blocks as are resident at once (two of 16 warps per SM); any count is correct
#define HIGGS_ENC(T, P) \
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, encode_pruned_kernel<T, P>, 512, smem) != cudaSuccess || per_sm < 1) per_sm = 1; \
    resident = (int64_t)per_sm * sm_count(); \
    blocks = (unsigned)(turns < resident ? turns : resident); \
    encode_pruned_kernel<T, P><<<blocks, 512, smem, st>>>(static_cast<const T*>(W), grid, d.n, tab, canonical, pk, fmt, bits, sc, d.N, d.K, d.rht_seed)
    int per_sm = 0;
    int64_t resident = 0;
    unsigned blocks = 0;
    if (w_dtype == HIGGS_F32 && d.p == 2) { HIGGS_ENC(float, 2); }
    else if (w_dtype == HIGGS_F32 && d.p == 1) { HIGGS_ENC(float, 1); }
    else if (w_dtype == HIGGS_BF16 && d.p == 2) { HIGGS_ENC(__nv_bfloat16, 2); }
    else if (w_dtype == HIGGS_BF16 && d.p == 1) { HIGGS_ENC(__nv_bfloat16, 1); }
    else return HIGGS_ERR_UNSUPPORTED;
#undef HIGGS_ENC
    *packed_done = packed != nullptr;
    return cuda_status(cudaGetLastError());
}

int launch_pack(const higgs_desc& d, const uint8_t* canonical, void* packed, cudaStream_t st) {
    const int64_t tiles = (d.N / 16) * (d.K / kGroup);
    if (tiles == 0) return HIGGS_OK;
    if (tiles > 0x7fffffff) return HIGGS_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(canonical) % 16) return HIGGS_ERR_INVALID_ARG;
    const Format f = format_of(d.p, d.n);
    if (f == Format::kNone) return HIGGS_ERR_UNSUPPORTED;
    uint32_t* out = static_cast<uint32_t*>(packed);
    if (d.p == 2) pack_kernel<2><<<(unsigned)tiles, 256, 0, st>>>(canonical, out, d.N, d.K, (int)f - 1, code_bits(d.n));
    else pack_kernel<1><<<(unsigned)tiles, 256, 0, st>>>(canonical, out, d.N, d.K, (int)f - 1, code_bits(d.n));
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
