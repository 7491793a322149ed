// Shared declarations of the HIGGS CUDA library (sm_100a only).
#pragma once

#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "higgs.h"

namespace higgs {

constexpr int kGroup = 1024;     // the only supported group size g
constexpr int kRowTile = 16;     // rows of W per mma tile (m16n8k16) and per scale tile
constexpr int kBlockK = 64;      // k-extent of one 512-byte packed block
constexpr int kMaxGather = 8;          // destinations of a gathered output (this device's own among them)
constexpr int kMaxGridDim = 4;        // grid fit and general encoder: 1 <= p <= 4
constexpr int kMaxGridPoints = 4096;  //                               n <= 4096 (64 KB of fp32 at p = 4)

// Output number m of the splitmix64 stream seeded with xi: 64 sign bits, for inputs 64 m .. 64 m + 63.
__host__ __device__ __forceinline__ uint64_t sign_word(uint64_t xi, uint64_t m) {
    uint64_t z = xi + (m + 1ull) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
// sign of input j: bit (j mod 64) of output floor(j / 64); 1 -> sign -1.
__host__ __device__ __forceinline__ uint32_t sign_bit(uint64_t xi, int64_t j) {
    return (uint32_t)((sign_word(xi, (uint64_t)j >> 6) >> ((uint64_t)j & 63ull)) & 1ull);
}

// How codes are stored in the packed stream.
//   kByteLut : one byte looks up one fp16x2 table entry (two consecutive k).
//              p=2,n=256: the byte is the code.  p=1,n=16: the byte holds the
//              codes of k (low nibble) and k+1 (high nibble).
//   kSixBit  : p=2,n=64: 6-bit codes, low nibbles and high bit-pairs in
//              separate planes (bit slices), see quantize.cu.
//   kNibble  : p=2,n=16: 4-bit codes, two per byte; the byte looks up an 8-byte
//              table entry (the fp16 pairs of both codes = two A-fragment registers).
//   kByte8   : p=1,n=256 (the constrained 8-bit grid): one byte = one input, a register takes two lookups.
enum class Format : int { kNone = 0, kByteLut = 1, kSixBit = 2, kNibble = 3, kByte8 = 4 };

__host__ __device__ inline Format format_of(int p, int n) {
    // a table index always covers two consecutive inputs: one p=2 code or two p=1 codes
    if (p == 2 && n == 256) return Format::kByteLut;
    if (p == 1 && n == 16) return Format::kByteLut;
    if (p == 2 && n == 64) return Format::kSixBit;
    if (p == 1 && n == 8) return Format::kSixBit;
    if (p == 2 && n == 16) return Format::kNibble;
    if (p == 1 && n == 4) return Format::kNibble;
    if (p == 1 && n == 256) return Format::kByte8;
    return Format::kNone;
}

// log2 of the grid size (bits per code)
__host__ __device__ inline int code_bits(int n) { int b = 0; while ((1 << b) < n) ++b; return b; }

// Validates the descriptor; returns HIGGS_OK or the error to hand back.
int check_desc(const higgs_desc* d);

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

inline int cuda_status(cudaError_t e) { return e == cudaSuccess ? HIGGS_OK : HIGGS_ERR_CUDA; }

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// One-time set-up per device (function attributes, occupancy queries) that several host threads may reach at once:
// `state[dev]` is read and written under one process-wide mutex.  Returns the stored value (0 = not yet set).
inline std::mutex& device_setup_mutex() { static std::mutex m; return m; }
template <typename F>
inline int device_once(int (&state)[64], F&& setup) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return setup();
    std::lock_guard<std::mutex> lock(device_setup_mutex());
    if (state[dev] == 0) state[dev] = setup();
    return state[dev];
}

// ---- programmatic dependent launch -----------------------------------------------------------
// Every kernel of the decode path is launched with the programmatic-stream-serialization
// attribute: it may start while the previous kernel of the stream is still running, does the work
// that depends on nothing (table build, weight prefetch) and then calls pdl_wait() before it
// touches anything the previous kernel may read or write.  pdl_trigger() lets the next kernel
// start as early as possible.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// The same with the blocks grouped into thread-block clusters of `cluster_x` along x.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                      unsigned cluster_x, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster_x;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---- in-register / warp-shuffle fast Walsh-Hadamard transform over 1024 ----
// A warp owns one group.  Lane l holds 32 values v[r], r = c*8 + e, standing
// for element index  idx = c*256 + l*8 + e  (c in 0..3, e in 0..7), so that a
// lane's four chunks are 8 consecutive elements each and a warp-wide chunk load
// is one contiguous 256-element run.  Butterflies over the e and c bits run in
// registers, the five lane bits through shfl.bfly.  The transform is the
// unnormalised Sylvester one (stages commute, so any bit order gives H v).
__device__ __forceinline__ void fwht1024_warp(float (&v)[32], int lane) {
#pragma unroll
    for (int h = 1; h < 32; h <<= 1) {
#pragma unroll
        for (int r = 0; r < 32; ++r) {
            if ((r & h) == 0) {
                float a = v[r], b = v[r | h];
                v[r] = a + b;
                v[r | h] = a - b;
            }
        }
    }
#pragma unroll
    for (int m = 1; m < 32; m <<= 1) {
        // upper lane of a pair: other - own, lower lane: own + other - one fused multiply-add with +-1 (exact product,
        // one rounding: the same value as the subtraction / addition)
        const float sgn = (lane & m) != 0 ? -1.0f : 1.0f;
#pragma unroll
        for (int r = 0; r < 32; ++r) {
            float o = __shfl_xor_sync(0xffffffffu, v[r], m);
            v[r] = fmaf(v[r], sgn, o);
        }
    }
}

// Flips the signs of the 32 values of this lane (mapping above) for the group starting at input k0 (a multiple
// of 1024): chunk c covers inputs k0 + c*256 + lane*8 .. +7, eight consecutive bits of one 64-bit sign word.
__device__ __forceinline__ void apply_signs1024(float (&v)[32], uint64_t xi, int64_t k0, int lane) {
    // the group's 16 sign words: lane l computes word l & 15, chunk c of a lane needs word 4c + lane/8
    const uint64_t word = sign_word(xi, ((uint64_t)k0 >> 6) + (uint64_t)(lane & 15));
    const uint32_t lo = (uint32_t)word, hi = (uint32_t)(word >> 32);
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const int src = 4 * c + (lane >> 3);
        const uint32_t from_lo = __shfl_sync(0xffffffffu, lo, src), from_hi = __shfl_sync(0xffffffffu, hi, src);
        const uint32_t bits = ((lane & 4) ? from_hi : from_lo) >> ((lane & 3) * 8);
#pragma unroll
        for (int e = 0; e < 8; ++e)
            v[c * 8 + e] = __uint_as_float(__float_as_uint(v[c * 8 + e]) ^ ((bits << (31 - e)) & 0x80000000u));
    }
}

// element index inside the group of register r of lane l (see above)
__device__ __forceinline__ int fwht_index(int lane, int r) { return (r >> 3) * 256 + lane * 8 + (r & 7); }

// ---- kernels' host-side launchers (defined in the .cu files) ---------------
int launch_rht_activations(const higgs_desc& d, const void* x, int64_t B, __half* xdag, float* zero_ptr,
                           size_t zero_floats, cudaStream_t st);
int launch_rht_debug(const higgs_desc& d, const void* x, int x_dtype, int64_t rows, float* out, int normalised,
                     cudaStream_t st);
// layers of at least this many (row, group) tasks are encoded with the pruned search
constexpr int64_t kPrunedMinTasks = 2048;
size_t encoder_table_bytes(int p);
int launch_encoder_table(int p, int n, const float* grid, void* table, cudaStream_t st);
int launch_encode(const higgs_desc& d, const void* W, int w_dtype, const float* grid, const void* table, void* build_space,
                  uint8_t* canonical, void* packed, void* scales, bool* packed_done, cudaStream_t st);
int launch_pack(const higgs_desc& d, const uint8_t* canonical, void* packed, cudaStream_t st);
int launch_unpack(const higgs_desc& d, const void* packed, uint8_t* canonical, cudaStream_t st);
int launch_dequantize(const higgs_desc& d, const uint8_t* canonical, const void* scales, const float* grid, void* W_out,
                      int w_dtype, cudaStream_t st);
// Further destinations of a product's output - the all-gather of a row-sharded layer fused into the epilogue: the same
// [B][ldy] window in the memory of other devices (peer-mapped pointers), written with plain stores.
struct GatherTargets {
    void* y[kMaxGather - 1];
    int count;
};
// Several matrices with the same K, grid and seed that read the same activations, run as one product over their
// concatenated rows (rows are independent in Appendix F's product): matrix i has rows[i] rows, its own packed stream,
// scales and output [B][rows[i]].
constexpr int kMaxMulti = 4;
struct MultiSegments {
    int count;
    int64_t rows[kMaxMulti];
    const void* packed[kMaxMulti];
    const void* scales[kMaxMulti];
    void* y[kMaxMulti];
};
// x_raw != nullptr: the activations as given (bf16); the kernel rotates them itself (only if linear_fused_eligible)
int launch_linear_mma(const higgs_desc& d, const __half* xdag, int64_t B, const void* packed, const void* scales,
                      const float* grid, void* y, int64_t ldy, int y_mode, cudaStream_t st, const void* x_raw = nullptr,
                      const GatherTargets* more = nullptr, __half* xdag_emit = nullptr, const MultiSegments* segs = nullptr);
int launch_scatter_out(const float* y32, int64_t B, int64_t N, void* const* dsts, int n_dst, int64_t ldy, int y_dtype,
                       cudaStream_t st);
bool linear_fused_eligible(const higgs_desc& d, int64_t B);
int launch_convert_out(const float* y32, void* y, int y_dtype, size_t count, cudaStream_t st);
size_t make_grid_workspace(int p, int n, int64_t m);
int launch_make_grid(int p, int n, const float* samples, int64_t m, int max_iters, float* grid_out, float* mse_out,
                     int32_t* iters_out, void* ws, cudaStream_t st);
int launch_layer_error(const higgs_desc& d, const uint8_t* canonical, const void* scales, const float* grid, const void* W,
                       int w_dtype, double* sums, cudaStream_t st);
int allocate_bits(int L, int J, const double* alpha, const double* t2, const int32_t* bits64, const int64_t* sizes,
                  int64_t budget64, int32_t* choice_out, double* objective_out);
int launch_encode_general(int p, int n, int64_t N, int64_t K, uint64_t xi, const void* W, int w_dtype, const float* grid,
                          uint16_t* codes, void* scales, double* sums, cudaStream_t st);
int launch_uniform_grid(int n, float* grid_out, float* step_out, float* mse_out, cudaStream_t st);
int linear_k_chunks(const higgs_desc& d, int64_t B);
bool linear_uses_atomics(const higgs_desc& d, int64_t B);   // K ranges meet in fp32 atomics: the output must be cleared first
// tensor-core path (B > 16)
bool tc_eligible(const higgs_desc& d, int64_t B);
size_t tc_workspace_bytes(const higgs_desc& d, int64_t B);
int tc_batch_tile(int64_t B);
int tc_k_split(const higgs_desc& d, int64_t B);
int launch_rht_tc(const higgs_desc& d, const void* x, int64_t B, __half* xdag_tc, cudaStream_t st);
int launch_linear_tc(const higgs_desc& d, const __half* xdag_tc, int64_t B, const void* packed, const void* scales,
                     const float* grid, void* y, int y_mode, cudaStream_t st, int64_t ldy = 0,
                     const GatherTargets* more = nullptr);
int read_tc_status(int clear);
int launch_error_ratio(double* sums, cudaStream_t st);
int read_grid_status(int clear);
int read_encode_status(int clear);
int launch_wait_selftest(uint32_t limit, int* result, cudaStream_t st);
int launch_tc_wait_selftest(uint32_t limit, int* result, cudaStream_t st);
int launch_stream_fence(cudaStream_t st);
int launch_reduce_slots(const float* slots, int world, int64_t count, void* y, int y_dtype, cudaStream_t st);
int launch_floor(int blocks, int threads, size_t smem, cudaStream_t st);
int launch_gaussian_samples(int p, uint64_t seed, int64_t m, float* out, cudaStream_t st);
int read_device_status(cudaStream_t st, int clear);

}  // namespace higgs
