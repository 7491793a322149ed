// C-ABI entry points: argument checking, workspace carving, kernel sequencing.
#include "common.cuh"

namespace higgs {

int check_desc(const higgs_desc* d) {
    if (!d) return HIGGS_ERR_INVALID_ARG;
    if (d->N < 0 || d->K < 0) return HIGGS_ERR_INVALID_ARG;
    if (d->g != kGroup) return HIGGS_ERR_UNSUPPORTED;
    if (format_of(d->p, d->n) == Format::kNone) return HIGGS_ERR_UNSUPPORTED;
    if (d->scale_dtype != HIGGS_F16) return HIGGS_ERR_UNSUPPORTED;
    if (d->layout_version != HIGGS_LAYOUT_VERSION) return HIGGS_ERR_UNSUPPORTED;
    if (d->N % kRowTile || d->K % kGroup) return HIGGS_ERR_UNSUPPORTED;
    if (d->N > (int64_t)1 << 30 || d->K > (int64_t)1 << 30) return HIGGS_ERR_UNSUPPORTED;
    return HIGGS_OK;
}

static bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace higgs

using namespace higgs;

extern "C" {

const char* higgs_status_string(int status) {
    switch (status) {
        case HIGGS_OK: return "ok";
        case HIGGS_ERR_INVALID_ARG: return "invalid argument";
        case HIGGS_ERR_UNSUPPORTED: return "unsupported (p, n, g, dtype, shape) combination";
        case HIGGS_ERR_WORKSPACE: return "workspace too small";
        case HIGGS_ERR_CUDA: return "CUDA runtime error";
        case HIGGS_ERR_TIMEOUT: return "bounded device-side wait ran out";
        case HIGGS_ERR_STATIC_SCRATCH: return "request exceeds the library's built-in scratch array";
        default: return "unknown status";
    }
}

int higgs_sign(uint64_t rht_seed, int64_t j) { return sign_bit(rht_seed, j) ? -1 : 1; }

size_t higgs_packed_bytes(const higgs_desc* d) {
    if (check_desc(d) != HIGGS_OK) return 0;
    const size_t pairs = (size_t)d->N * (size_t)d->K / 2;
    const Format f = format_of(d->p, d->n);
    return f == Format::kSixBit ? pairs / 4 * 3 : f == Format::kNibble ? pairs / 2 : f == Format::kByte8 ? pairs * 2 : pairs;
}

size_t higgs_scales_bytes(const higgs_desc* d) {
    if (check_desc(d) != HIGGS_OK) return 0;
    return (size_t)d->N * (size_t)(d->K / d->g) * 2;
}

size_t higgs_canonical_bytes(const higgs_desc* d) {
    if (check_desc(d) != HIGGS_OK) return 0;
    return (size_t)d->N * (size_t)d->K / (size_t)d->p;
}

size_t higgs_workspace_bytes(const higgs_desc* d, int op, int64_t B) {
    if (!d) return 0;
    if (op == HIGGS_OP_MAKE_GRID) {
        if (!(d->p >= 1 && d->p <= kMaxGridDim && d->n >= 1 && d->n <= kMaxGridPoints && d->K >= d->n)) return 0;
        return make_grid_workspace(d->p, d->n, d->K);
    }
    if (op == HIGGS_OP_MAKE_GRID_SEEDED) {
        if (!(d->p >= 1 && d->p <= kMaxGridDim && d->n >= 1 && d->n <= kMaxGridPoints && d->K >= d->n)) return 0;
        return align_up(make_grid_workspace(d->p, d->n, d->K), 256) + (size_t)d->K * d->p * sizeof(float);
    }
    if (check_desc(d) != HIGGS_OK) return 0;
    if (op == HIGGS_OP_QUANTIZE) return align_up(higgs_canonical_bytes(d), 256) + 256;
    if (op == HIGGS_OP_LINEAR) {
        if (B < 1) return 0;
        const size_t stream_path = align_up((size_t)B * d->K * 2, 256) + align_up((size_t)B * d->N * 4, 256) + 256;
        const size_t tc_path = tc_eligible(*d, B) ? align_up(tc_workspace_bytes(*d, B), 256) + 256 : 0;
        return stream_path > tc_path ? stream_path : tc_path;
    }
    return 0;
}

int higgs_make_grid(int p, int n, const float* samples, int64_t num_samples, int max_iters, float* grid_out,
                    float* mse_out, int32_t* iters_out, void* workspace, size_t workspace_bytes, void* stream) {
    if (!samples || !grid_out || !workspace || max_iters < 1) return HIGGS_ERR_INVALID_ARG;
    if (p < 1 || p > kMaxGridDim || n < 1 || n > kMaxGridPoints) return HIGGS_ERR_UNSUPPORTED;
    if (num_samples < n || num_samples > ((int64_t)1 << 31) - 1) return HIGGS_ERR_INVALID_ARG;
    if (!aligned(workspace, 256)) return HIGGS_ERR_INVALID_ARG;
    if (workspace_bytes < make_grid_workspace(p, n, num_samples)) return HIGGS_ERR_WORKSPACE;
    const int rc = launch_make_grid(p, n, samples, num_samples, max_iters, grid_out, mse_out, iters_out, workspace,
                                    as_stream(stream));
    return rc != HIGGS_OK ? rc : launch_stream_fence(as_stream(stream));
}

int higgs_make_grid_seeded(int p, int n, uint64_t sample_seed, int log2_samples, int max_iters, float* grid_out,
                            float* mse_out, int32_t* iters_out, void* workspace, size_t workspace_bytes, void* stream) {
    if (!grid_out || !workspace || max_iters < 1) return HIGGS_ERR_INVALID_ARG;
    if (p < 1 || p > kMaxGridDim || n < 1 || n > kMaxGridPoints) return HIGGS_ERR_UNSUPPORTED;
    if (log2_samples < 1 || log2_samples > 24 || ((int64_t)1 << log2_samples) < n) return HIGGS_ERR_INVALID_ARG;
    if (!aligned(workspace, 256)) return HIGGS_ERR_INVALID_ARG;
    const int64_t m = (int64_t)1 << log2_samples;
    const size_t fit = align_up(make_grid_workspace(p, n, m), 256);
    if (workspace_bytes < fit + (size_t)m * p * sizeof(float)) return HIGGS_ERR_WORKSPACE;
    float* samples = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + fit);
    const int rc = launch_gaussian_samples(p, sample_seed, m, samples, as_stream(stream));
    if (rc != HIGGS_OK) return rc;
    const int rc2 = launch_make_grid(p, n, samples, m, max_iters, grid_out, mse_out, iters_out, workspace, as_stream(stream));
    return rc2 != HIGGS_OK ? rc2 : launch_stream_fence(as_stream(stream));
}

int higgs_gaussian_samples(int p, uint64_t sample_seed, int64_t num_samples, float* samples_out, void* stream) {
    if (p < 1 || p > kMaxGridDim || num_samples < 0 || num_samples > ((int64_t)1 << 28)) return HIGGS_ERR_INVALID_ARG;
    if (num_samples == 0) return HIGGS_OK;
    if (!samples_out) return HIGGS_ERR_INVALID_ARG;
    return launch_gaussian_samples(p, sample_seed, num_samples, samples_out, as_stream(stream));
}

int higgs_shard_rows(int64_t N, int32_t world, int32_t rank, int32_t multiple, int64_t* begin_out, int64_t* count_out) {
    if (!begin_out || !count_out || world < 1 || rank < 0 || rank >= world || multiple < kRowTile || multiple % kRowTile)
        return HIGGS_ERR_INVALID_ARG;
    if (N < 0 || N % multiple) return HIGGS_ERR_UNSUPPORTED;
    const int64_t units = N / multiple, base = units / world, extra = units % world;
    const int64_t begin = rank * base + (rank < extra ? rank : extra);
    *begin_out = begin * multiple;
    *count_out = (base + (rank < extra ? 1 : 0)) * multiple;
    return HIGGS_OK;
}

uint64_t higgs_shard_seed(uint64_t rht_seed, int64_t k_offset) {
    // output number m + k_offset / 64 of the stream seeded with xi is output number m of the stream seeded with
    // xi + (k_offset / 64) * golden-ratio increment: the sign function's state advances by that increment per output
    return rht_seed + (uint64_t)(k_offset / 64) * 0x9E3779B97F4A7C15ull;
}

int higgs_linear_kshard(const higgs_desc* d, const void* x_shard, int64_t B, const void* packed, const void* scales,
                        const float* grid, void* const* slot_bufs, int32_t world, int32_t rank, void* workspace,
                        size_t workspace_bytes, void* stream) {
    if (!d || !slot_bufs || world < 1 || world > kMaxGather || rank < 0 || rank >= world || B < 0) return HIGGS_ERR_INVALID_ARG;
    void* dst[kMaxGather];
    for (int i = 0; i < world; ++i) {
        if (!slot_bufs[i]) return HIGGS_ERR_INVALID_ARG;
        dst[i] = static_cast<float*>(slot_bufs[i]) + (size_t)rank * (size_t)B * (size_t)d->N;    // slot `rank` of device i
    }
    // the own device's buffer first (slot_bufs[rank]), then the peers' in rank order
    void* ordered[kMaxGather];
    int n = 0;
    ordered[n++] = dst[rank];
    for (int i = 0; i < world; ++i)
        if (i != rank) ordered[n++] = dst[i];
    return higgs_linear_gather(d, x_shard, B, packed, scales, grid, ordered, world, d->N, 0, HIGGS_F32, workspace, workspace_bytes,
                               stream);
}

int higgs_reduce_slots(const float* slots, int32_t world, int64_t count, void* y, int y_dtype, void* stream) {
    if (world < 1 || world > kMaxGather || count < 0 || count % 4) return HIGGS_ERR_INVALID_ARG;
    if (y_dtype != HIGGS_F32 && y_dtype != HIGGS_BF16) return HIGGS_ERR_UNSUPPORTED;
    if (count == 0) return HIGGS_OK;
    if (!slots || !y || !aligned(slots, 16) || !aligned(y, 16)) return HIGGS_ERR_INVALID_ARG;
    return launch_reduce_slots(slots, world, count, y, y_dtype, as_stream(stream));
}

int higgs_launch_floor(int32_t blocks, int32_t threads, size_t shared_bytes, void* stream) {
    if (blocks < 1 || threads < 1 || threads > 1024 || shared_bytes > 232448) return HIGGS_ERR_INVALID_ARG;
    return launch_floor(blocks, threads, shared_bytes, as_stream(stream));
}

int higgs_selftest_wait(int32_t which, uint32_t polls, int32_t* result_out, void* stream) {
    if (!result_out || polls > (1u << 20)) return HIGGS_ERR_INVALID_ARG;
    if (which == 0) return launch_wait_selftest(polls, result_out, as_stream(stream));
    if (which == 1) return launch_tc_wait_selftest(polls, result_out, as_stream(stream));
    return HIGGS_ERR_INVALID_ARG;
}

int higgs_general_tuples(int p) { return p >= 1 && p <= kMaxGridDim ? (kGroup + p - 1) / p : 0; }

int higgs_quantize_general(int p, int n, int64_t N, int64_t K, uint64_t rht_seed, const void* W, int w_dtype,
                           const float* grid, uint16_t* codes_out, void* scales_out, double* sums_out, void* stream) {
    if (p < 1 || p > kMaxGridDim || n < 1 || n > kMaxGridPoints) return HIGGS_ERR_UNSUPPORTED;
    if (w_dtype != HIGGS_F32 && w_dtype != HIGGS_BF16) return HIGGS_ERR_UNSUPPORTED;
    if (N < 0 || K < 0) return HIGGS_ERR_INVALID_ARG;
    if (K % kGroup) return HIGGS_ERR_UNSUPPORTED;
    if (N == 0 || K == 0) return HIGGS_OK;
    if (!W || !grid || !codes_out || !scales_out) return HIGGS_ERR_INVALID_ARG;
    if (!aligned(W, 16) || !aligned(codes_out, 2) || !aligned(scales_out, 2) || (sums_out && !aligned(sums_out, 8)))
        return HIGGS_ERR_INVALID_ARG;
    const int rc = launch_encode_general(p, n, N, K, rht_seed, W, w_dtype, grid, codes_out, scales_out, sums_out,
                                         as_stream(stream));
    return rc != HIGGS_OK || !sums_out ? rc : launch_error_ratio(sums_out, as_stream(stream));
}

int higgs_make_uniform_grid(int n, float* grid_out, float* step_out, float* mse_out, void* stream) {
    if (!grid_out) return HIGGS_ERR_INVALID_ARG;
    if (n < 2 || n > 256) return HIGGS_ERR_UNSUPPORTED;
    const int rc = launch_uniform_grid(n, grid_out, step_out, mse_out, as_stream(stream));
    return rc != HIGGS_OK ? rc : launch_stream_fence(as_stream(stream));
}

size_t higgs_encoder_table_bytes(int p, int n) {
    return format_of(p, n) == Format::kNone ? 0 : encoder_table_bytes(p);
}

int higgs_make_encoder_table(int p, int n, const float* grid, void* table_out, void* stream) {
    if (format_of(p, n) == Format::kNone) return HIGGS_ERR_UNSUPPORTED;
    if (!grid || !table_out || !aligned(table_out, 16)) return HIGGS_ERR_INVALID_ARG;
    const int rc = launch_encoder_table(p, n, grid, table_out, as_stream(stream));
    return rc != HIGGS_OK ? rc : launch_stream_fence(as_stream(stream));
}

int higgs_quantize_prepared(const higgs_desc* d, const void* W, int w_dtype, const float* grid, const void* table,
                            void* packed_out, void* scales_out, uint8_t* canonical_out, void* workspace,
                            size_t workspace_bytes, void* stream) {
    int rc = check_desc(d);
    if (rc != HIGGS_OK) return rc;
    if (w_dtype != HIGGS_F32 && w_dtype != HIGGS_BF16) return HIGGS_ERR_UNSUPPORTED;
    if (d->N == 0 || d->K == 0) return HIGGS_OK;
    if (!W || !grid || !packed_out || !scales_out) return HIGGS_ERR_INVALID_ARG;
    if (!aligned(W, 16) || !aligned(packed_out, 16) || !aligned(scales_out, 16) || (table && !aligned(table, 16)))
        return HIGGS_ERR_INVALID_ARG;
    if (canonical_out && !aligned(canonical_out, 16)) return HIGGS_ERR_INVALID_ARG;
    if (workspace && !aligned(workspace, 256)) return HIGGS_ERR_INVALID_ARG;
    if (!canonical_out) {
        if (!workspace) return HIGGS_ERR_INVALID_ARG;
        if (workspace_bytes < higgs_workspace_bytes(d, HIGGS_OP_QUANTIZE, 0)) return HIGGS_ERR_WORKSPACE;
    }
    cudaStream_t st = as_stream(stream);
    // The workspace holds the cell table of a large layer (whose search kernel emits the packed stream itself and needs
    // no canonical copy) or the canonical codes of a small one (exhaustive scan, then the pack kernel) - never both.
    // Without a workspace (the caller wants the canonical codes and lends none) the table of a large layer is built in
    // the packed output, which only the pack kernel writes, after the encoder has finished.
    const bool ws_table = workspace && workspace_bytes >= encoder_table_bytes(d->p);
    void* build_space = table ? nullptr : (ws_table ? workspace : packed_out);
    const bool fuse = table || ws_table;
    uint8_t* canonical = canonical_out ? canonical_out : static_cast<uint8_t*>(workspace);
    // (a small layer ignores the table arguments; a large one ignores `canonical` when it is the workspace)
    bool packed_done = false;
    const int64_t tasks = d->N * (d->K / kGroup);
    const bool large = tasks >= kPrunedMinTasks;
    rc = launch_encode(*d, W, w_dtype, grid, table, build_space, large ? canonical_out : canonical,
                       (large && fuse) ? packed_out : nullptr, scales_out, &packed_done, st);
    if (rc != HIGGS_OK) return rc;
    if (!packed_done) {
        rc = launch_pack(*d, large ? canonical_out : canonical, packed_out, st);
        if (rc != HIGGS_OK) return rc;
    }
    return launch_stream_fence(st);
}

int higgs_quantize(const higgs_desc* d, const void* W, int w_dtype, const float* grid, void* packed_out,
                   void* scales_out, uint8_t* canonical_out, void* workspace, size_t workspace_bytes, void* stream) {
    return higgs_quantize_prepared(d, W, w_dtype, grid, nullptr, packed_out, scales_out, canonical_out, workspace,
                                   workspace_bytes, stream);
}

int higgs_dequantize(const higgs_desc* d, const void* packed, const void* scales, const float* grid, void* W_out,
                     int w_dtype, void* workspace, size_t workspace_bytes, void* stream) {
    int rc = check_desc(d);
    if (rc != HIGGS_OK) return rc;
    if (w_dtype != HIGGS_F32 && w_dtype != HIGGS_BF16) return HIGGS_ERR_UNSUPPORTED;
    if (d->N == 0 || d->K == 0) return HIGGS_OK;
    if (!packed || !scales || !grid || !W_out || !workspace) return HIGGS_ERR_INVALID_ARG;
    if (!aligned(packed, 16) || !aligned(scales, 16) || !aligned(W_out, 16) || !aligned(workspace, 256)) return HIGGS_ERR_INVALID_ARG;
    if (workspace_bytes < higgs_workspace_bytes(d, HIGGS_OP_QUANTIZE, 0)) return HIGGS_ERR_WORKSPACE;
    cudaStream_t st = as_stream(stream);
    uint8_t* canonical = static_cast<uint8_t*>(workspace);
    rc = launch_unpack(*d, packed, canonical, st);
    if (rc != HIGGS_OK) return rc;
    return launch_dequantize(*d, canonical, scales, grid, W_out, w_dtype, st);
}

int higgs_layer_error(const higgs_desc* d, const void* W, int w_dtype, const void* packed, const void* scales,
                      const float* grid, double* sums_out, void* workspace, size_t workspace_bytes, void* stream) {
    int rc = check_desc(d);
    if (rc != HIGGS_OK) return rc;
    if (w_dtype != HIGGS_F32 && w_dtype != HIGGS_BF16) return HIGGS_ERR_UNSUPPORTED;
    if (!sums_out || !aligned(sums_out, 8)) return HIGGS_ERR_INVALID_ARG;
    if (d->N == 0 || d->K == 0) return cuda_status(cudaMemsetAsync(sums_out, 0, 3 * sizeof(double), as_stream(stream)));
    if (!W || !packed || !scales || !grid || !workspace) return HIGGS_ERR_INVALID_ARG;
    if (!aligned(W, 16) || !aligned(packed, 16) || !aligned(scales, 16) || !aligned(workspace, 256)) return HIGGS_ERR_INVALID_ARG;
    if (workspace_bytes < higgs_workspace_bytes(d, HIGGS_OP_QUANTIZE, 0)) return HIGGS_ERR_WORKSPACE;
    cudaStream_t st = as_stream(stream);
    uint8_t* canonical = static_cast<uint8_t*>(workspace);
    rc = launch_unpack(*d, packed, canonical, st);
    if (rc != HIGGS_OK) return rc;
    rc = launch_layer_error(*d, canonical, scales, grid, W, w_dtype, sums_out, st);
    return rc != HIGGS_OK ? rc : launch_error_ratio(sums_out, st);
}

int higgs_allocate_bits(int32_t num_layers, int32_t num_options, const double* alpha, const double* t2, const int32_t* bits64,
                        const int64_t* sizes, int64_t budget64, int32_t* choice_out, double* objective_out) {
    return allocate_bits(num_layers, num_options, alpha, t2, bits64, sizes, budget64, choice_out, objective_out);
}

int higgs_rotate_activations(const higgs_desc* d, const void* x, int64_t B, void* xdag_out, void* stream) {
    int rc = check_desc(d);
    if (rc != HIGGS_OK) return rc;
    if (B < 0) return HIGGS_ERR_INVALID_ARG;
    if (B == 0 || d->K == 0) return HIGGS_OK;
    if (!x || !xdag_out || !aligned(x, 16) || !aligned(xdag_out, 16)) return HIGGS_ERR_INVALID_ARG;
    if (tc_eligible(*d, B)) return launch_rht_tc(*d, x, B, static_cast<__half*>(xdag_out), as_stream(stream));
    return launch_rht_activations(*d, x, B, static_cast<__half*>(xdag_out), nullptr, 0, as_stream(stream));
}

// Shared tail of higgs_linear / higgs_linear_prerotated: D2-D5 on rotated activations.
static int linear_tail(const higgs_desc* d, const __half* xdag, int64_t B, const void* packed, const void* scales,
                       const float* grid, void* y, int y_dtype, float* y32, bool target_is_clear, cudaStream_t st) {
    const bool split = linear_uses_atomics(*d, B);
    float* acc_target = split ? (y_dtype == HIGGS_F32 ? static_cast<float*>(y) : y32) : nullptr;
    if (split && !target_is_clear) {
        if (cudaMemsetAsync(acc_target, 0, (size_t)B * d->N * sizeof(float), st) != cudaSuccess) return HIGGS_ERR_CUDA;
    }
    for (int64_t b0 = 0; b0 < B; b0 += 16) {
        const int64_t bn = B - b0 < 16 ? B - b0 : 16;
        void* yo;
        int mode;
        if (split) { yo = acc_target + b0 * d->N; mode = 2; }
        else if (y_dtype == HIGGS_F32) { yo = static_cast<float*>(y) + b0 * d->N; mode = 0; }
        else { yo = static_cast<__nv_bfloat16*>(y) + b0 * d->N; mode = 1; }
        int rc = launch_linear_mma(*d, xdag + b0 * d->K, bn, packed, scales, grid, yo, d->N, mode, st);
        if (rc != HIGGS_OK) return rc;
    }
    if (split && y_dtype == HIGGS_BF16) return launch_convert_out(y32, y, y_dtype, (size_t)B * d->N, st);
    return HIGGS_OK;
}

static int linear_args(const higgs_desc* d, int64_t B, const void* x, const void* packed, const void* scales,
                       const float* grid, void* y, int y_dtype, void* workspace, size_t workspace_bytes) {
    int rc = check_desc(d);
    if (rc != HIGGS_OK) return rc;
    if (y_dtype != HIGGS_F32 && y_dtype != HIGGS_BF16) return HIGGS_ERR_UNSUPPORTED;
    if (B < 0) return HIGGS_ERR_INVALID_ARG;
    if (B == 0 || d->N == 0) return -1;   // nothing to do
    if (d->K == 0) return HIGGS_ERR_UNSUPPORTED;
    if (!x || !packed || !scales || !grid || !y || !workspace) return HIGGS_ERR_INVALID_ARG;
    if (!aligned(x, 16) || !aligned(packed, 16) || !aligned(scales, 16) || !aligned(workspace, 256) || !aligned(y, 16))
        return HIGGS_ERR_INVALID_ARG;
    if (workspace_bytes < higgs_workspace_bytes(d, HIGGS_OP_LINEAR, B)) return HIGGS_ERR_WORKSPACE;
    return HIGGS_OK;
}

int higgs_linear(const higgs_desc* d, const void* x, int64_t B, const void* packed, const void* scales,
                 const float* grid, void* y, int y_dtype, void* workspace, size_t workspace_bytes, void* stream) {
    int rc = linear_args(d, B, x, packed, scales, grid, y, y_dtype, workspace, workspace_bytes);
    if (rc != HIGGS_OK) return rc < 0 ? HIGGS_OK : rc;
    cudaStream_t st = as_stream(stream);
    if (tc_eligible(*d, B)) {
        // dense-contraction regime: rotate into the blocked operand layout, then one tcgen05 pass over the codes
        rc = launch_rht_tc(*d, x, B, static_cast<__half*>(workspace), st);
        if (rc != HIGGS_OK) return rc;
        return launch_linear_tc(*d, static_cast<const __half*>(workspace), B, packed, scales, grid, y,
                                y_dtype == HIGGS_F32 ? 0 : 1, st);
    }
    if (linear_fused_eligible(*d, B)) {
        // one or two tokens, K not split: the product kernel rotates the activations itself (D1 fused into D2-D5)
        void* yo = y;
        return launch_linear_mma(*d, nullptr, B, packed, scales, grid, yo, d->N, y_dtype == HIGGS_F32 ? 0 : 1, st, x);
    }
    __half* xdag = static_cast<__half*>(workspace);
    float* y32 = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + align_up((size_t)B * d->K * 2, 256));
    const bool split = linear_uses_atomics(*d, B);
    float* acc_target = split ? (y_dtype == HIGGS_F32 ? static_cast<float*>(y) : y32) : nullptr;
    // D1: rotate the activations once (and clear the accumulation target of a K-split product)
    rc = launch_rht_activations(*d, x, B, xdag, acc_target, split ? (size_t)B * d->N : 0, st);
    if (rc != HIGGS_OK) return rc;
    // D2-D5: stream codes, look up, contract, reduce
    return linear_tail(d, xdag, B, packed, scales, grid, y, y_dtype, y32, true, st);
}

int higgs_linear_share(const higgs_desc* d, const void* x, int64_t B, const void* packed, const void* scales,
                       const float* grid, void* y, int y_dtype, void* xdag_out, void* workspace, size_t workspace_bytes,
                       void* stream) {
    int rc = linear_args(d, B, x, packed, scales, grid, y, y_dtype, workspace, workspace_bytes);
    if (rc != HIGGS_OK) return rc < 0 ? HIGGS_OK : rc;
    if (!xdag_out || !aligned(xdag_out, 16)) return HIGGS_ERR_INVALID_ARG;
    cudaStream_t st = as_stream(stream);
    if (!tc_eligible(*d, B) && linear_fused_eligible(*d, B))
        // one launch: the product kernel rotates x itself and its first block leaves x+ behind for the other layers
        return launch_linear_mma(*d, nullptr, B, packed, scales, grid, y, d->N, y_dtype == HIGGS_F32 ? 0 : 1, st, x, nullptr,
                                 static_cast<__half*>(xdag_out));
    rc = higgs_rotate_activations(d, x, B, xdag_out, stream);
    if (rc != HIGGS_OK) return rc;
    return higgs_linear_prerotated(d, xdag_out, B, packed, scales, grid, y, y_dtype, workspace, workspace_bytes, stream);
}

size_t higgs_linear_multi_workspace_bytes(int32_t count, const higgs_desc* const* descs, int64_t B) {
    if (count < 1 || count > kMaxMulti || !descs || !descs[0]) return 0;
    higgs_desc v = *descs[0];
    size_t most = 0;
    v.N = 0;
    for (int i = 0; i < count; ++i) {
        if (!descs[i]) return 0;
        v.N += descs[i]->N;
        const size_t one = higgs_workspace_bytes(descs[i], HIGGS_OP_LINEAR, B);
        if (one == 0 && descs[i]->N != 0) return 0;
        most = one > most ? one : most;
    }
    const size_t all = higgs_workspace_bytes(&v, HIGGS_OP_LINEAR, B);
    return all > most ? all : most;
}

int higgs_linear_multi(int32_t count, const higgs_desc* const* descs, const void* x, int64_t B, const void* const* packed,
                       const void* const* scales, const float* grid, void* const* ys, int y_dtype, void* workspace,
                       size_t workspace_bytes, void* stream) {
    if (count < 1 || count > kMaxMulti || !descs || !packed || !scales || !ys) return HIGGS_ERR_INVALID_ARG;
    if (y_dtype != HIGGS_F32 && y_dtype != HIGGS_BF16) return HIGGS_ERR_UNSUPPORTED;
    if (B < 0) return HIGGS_ERR_INVALID_ARG;
    higgs_desc v;
    MultiSegments segs;
    segs.count = 0;
    for (int i = 0; i < count; ++i) {
        const higgs_desc* d = descs[i];
        const int rc = check_desc(d);
        if (rc != HIGGS_OK) return rc;
        if (i == 0) { v = *d; v.N = 0; }
        else if (d->p != v.p || d->n != v.n || d->g != v.g || d->K != v.K || d->rht_seed != v.rht_seed) return HIGGS_ERR_INVALID_ARG;
        if (d->N == 0) continue;
        if (!packed[i] || !scales[i] || !ys[i] || !aligned(packed[i], 16) || !aligned(scales[i], 16) || !aligned(ys[i], 16))
            return HIGGS_ERR_INVALID_ARG;
        segs.rows[segs.count] = d->N;
        segs.packed[segs.count] = packed[i];
        segs.scales[segs.count] = scales[i];
        segs.y[segs.count] = ys[i];
        ++segs.count;
        v.N += d->N;
    }
    if (B == 0 || v.N == 0) return HIGGS_OK;
    if (v.K == 0) return HIGGS_ERR_UNSUPPORTED;
    if (!x || !grid || !workspace || !aligned(x, 16) || !aligned(workspace, 256)) return HIGGS_ERR_INVALID_ARG;
    if (workspace_bytes < higgs_linear_multi_workspace_bytes(count, descs, B)) return HIGGS_ERR_WORKSPACE;
    cudaStream_t st = as_stream(stream);
    const int mode = y_dtype == HIGGS_F32 ? 0 : 1;
    if (segs.count > 1 && B <= 16 && !tc_eligible(v, B) && !linear_uses_atomics(v, B)) {
        // ONE launch of the small-batch kernel over the concatenated rows (per 16 tokens), the rotation done once
        if (linear_fused_eligible(v, B))
            return launch_linear_mma(v, nullptr, B, segs.packed[0], segs.scales[0], grid, segs.y[0], segs.rows[0], mode, st, x,
                                     nullptr, nullptr, &segs);
        __half* xdag = static_cast<__half*>(workspace);
        int rc = launch_rht_activations(v, x, B, xdag, nullptr, 0, st);
        if (rc != HIGGS_OK) return rc;
        const size_t esz = y_dtype == HIGGS_F32 ? 4 : 2;
        for (int64_t b0 = 0; b0 < B; b0 += 16) {
            const int64_t bn = B - b0 < 16 ? B - b0 : 16;
            MultiSegments part = segs;
            for (int i = 0; i < segs.count; ++i) part.y[i] = static_cast<uint8_t*>(segs.y[i]) + (size_t)b0 * segs.rows[i] * esz;
            rc = launch_linear_mma(v, xdag + b0 * v.K, bn, part.packed[0], part.scales[0], grid, part.y[0], part.rows[0], mode, st,
                                   nullptr, nullptr, nullptr, &part);
            if (rc != HIGGS_OK) return rc;
        }
        return HIGGS_OK;
    }
    // other shapes and batches (tensor-core path, K ranges that meet in atomics): one higgs_linear per matrix
    for (int i = 0; i < count; ++i) {
        if (descs[i]->N == 0) continue;
        const int rc = higgs_linear(descs[i], x, B, packed[i], scales[i], grid, ys[i], y_dtype, workspace, workspace_bytes, stream);
        if (rc != HIGGS_OK) return rc;
    }
    return HIGGS_OK;
}

int higgs_linear_multi_launch_count(int32_t count, const higgs_desc* const* descs, int64_t B, int y_dtype) {
    if (count < 1 || count > kMaxMulti || !descs || B < 1) return 0;
    higgs_desc v = *descs[0];
    v.N = 0;
    int live = 0, separate = 0;
    for (int i = 0; i < count; ++i) {
        if (check_desc(descs[i]) != HIGGS_OK) return 0;
        if (descs[i]->N == 0) continue;
        v.N += descs[i]->N;
        ++live;
        separate += higgs_linear_launch_count(descs[i], B, y_dtype);
    }
    if (live > 1 && B <= 16 && !tc_eligible(v, B) && !linear_uses_atomics(v, B))
        return linear_fused_eligible(v, B) ? 1 : 1 + (int)((B + 15) / 16);
    return separate;
}

int higgs_linear_gather(const higgs_desc* d, const void* x, int64_t B, const void* packed, const void* scales,
                        const float* grid, void* const* y_dsts, int32_t n_dst, int64_t ld, int64_t row_offset, int y_dtype,
                        void* workspace, size_t workspace_bytes, void* stream) {
    if (!y_dsts || n_dst < 1 || n_dst > kMaxGather) return HIGGS_ERR_INVALID_ARG;
    int rc = linear_args(d, B, x, packed, scales, grid, y_dsts[0], y_dtype, workspace, workspace_bytes);
    if (rc != HIGGS_OK) return rc < 0 ? HIGGS_OK : rc;
    if (row_offset < 0 || row_offset % kRowTile || ld < row_offset + d->N || ld % 8) return HIGGS_ERR_INVALID_ARG;
    const size_t esz = y_dtype == HIGGS_F32 ? 4 : 2;
    void* dst[kMaxGather];
    for (int i = 0; i < n_dst; ++i) {
        if (!y_dsts[i] || !aligned(y_dsts[i], 16)) return HIGGS_ERR_INVALID_ARG;
        dst[i] = static_cast<uint8_t*>(y_dsts[i]) + (size_t)row_offset * esz;       // this shard's columns of [B][ld]
    }
    GatherTargets more;
    more.count = n_dst - 1;
    for (int i = 0; i < kMaxGather - 1; ++i) more.y[i] = i + 1 < n_dst ? dst[i + 1] : nullptr;
    cudaStream_t st = as_stream(stream);
    const int mode = y_dtype == HIGGS_F32 ? 0 : 1;
    if (tc_eligible(*d, B)) {
        rc = launch_rht_tc(*d, x, B, static_cast<__half*>(workspace), st);
        if (rc != HIGGS_OK) return rc;
        return launch_linear_tc(*d, static_cast<const __half*>(workspace), B, packed, scales, grid, dst[0], mode, st, ld, &more);
    }
    if (linear_fused_eligible(*d, B))
        return launch_linear_mma(*d, nullptr, B, packed, scales, grid, dst[0], ld, mode, st, x, &more);
    __half* xdag = static_cast<__half*>(workspace);
    float* y32 = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + align_up((size_t)B * d->K * 2, 256));
    const bool split = linear_uses_atomics(*d, B);
    // D1 (and, for a K-split product, the cleared contiguous fp32 accumulator in the workspace)
    rc = launch_rht_activations(*d, x, B, xdag, split ? y32 : nullptr, split ? (size_t)B * d->N : 0, st);
    if (rc != HIGGS_OK) return rc;
    for (int64_t b0 = 0; b0 < B; b0 += 16) {
        const int64_t bn = B - b0 < 16 ? B - b0 : 16;
        if (split) {
            rc = launch_linear_mma(*d, xdag + b0 * d->K, bn, packed, scales, grid, y32 + b0 * d->N, d->N, 2, st);
        } else {
            GatherTargets m2 = more;
            for (int i = 0; i < more.count; ++i) m2.y[i] = static_cast<uint8_t*>(more.y[i]) + (size_t)b0 * ld * esz;
            rc = launch_linear_mma(*d, xdag + b0 * d->K, bn, packed, scales, grid,
                                   static_cast<uint8_t*>(dst[0]) + (size_t)b0 * ld * esz, ld, mode, st, nullptr, &m2);
        }
        if (rc != HIGGS_OK) return rc;
    }
    // a K-split product sums with atomics into its own contiguous buffer; one small kernel spreads the result
    if (split) return launch_scatter_out(y32, B, d->N, dst, n_dst, ld, y_dtype, st);
    return HIGGS_OK;
}

int higgs_linear_prerotated(const higgs_desc* d, const void* xdag, int64_t B, const void* packed, const void* scales,
                            const float* grid, void* y, int y_dtype, void* workspace, size_t workspace_bytes,
                            void* stream) {
    int rc = linear_args(d, B, xdag, packed, scales, grid, y, y_dtype, workspace, workspace_bytes);
    if (rc != HIGGS_OK) return rc < 0 ? HIGGS_OK : rc;
    if (tc_eligible(*d, B))
        return launch_linear_tc(*d, static_cast<const __half*>(xdag), B, packed, scales, grid, y,
                                y_dtype == HIGGS_F32 ? 0 : 1, as_stream(stream));
    float* y32 = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + align_up((size_t)B * d->K * 2, 256));
    return linear_tail(d, static_cast<const __half*>(xdag), B, packed, scales, grid, y, y_dtype, y32, false,
                       as_stream(stream));
}

int higgs_linear_host(const higgs_desc* d, const void* x_host, int64_t B, const void* packed, const void* scales,
                      const float* grid, void* y_host, int y_dtype, void* workspace, size_t workspace_bytes,
                      void* stream) {
    int rc = check_desc(d);
    if (rc != HIGGS_OK) return rc;
    if (y_dtype != HIGGS_F32 && y_dtype != HIGGS_BF16) return HIGGS_ERR_UNSUPPORTED;
    if (B < 0) return HIGGS_ERR_INVALID_ARG;
    if (B == 0 || d->N == 0) return HIGGS_OK;
    if (!x_host || !y_host || !workspace || !aligned(workspace, 256)) return HIGGS_ERR_INVALID_ARG;
    const size_t inner = higgs_workspace_bytes(d, HIGGS_OP_LINEAR, B);
    const size_t xb = align_up((size_t)B * d->K * 2, 256);
    const size_t yb = align_up((size_t)B * d->N * (y_dtype == HIGGS_F32 ? 4 : 2), 256);
    if (workspace_bytes < inner + xb + yb) return HIGGS_ERR_WORKSPACE;
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    void* x_dev = ws + inner;
    void* y_dev = ws + inner + xb;
    cudaStream_t st = as_stream(stream);
    if (cudaMemcpyAsync(x_dev, x_host, (size_t)B * d->K * 2, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return HIGGS_ERR_CUDA;
    rc = higgs_linear(d, x_dev, B, packed, scales, grid, y_dev, y_dtype, workspace, inner, stream);
    if (rc != HIGGS_OK) return rc;
    if (cudaMemcpyAsync(y_host, y_dev, (size_t)B * d->N * (y_dtype == HIGGS_F32 ? 4 : 2), cudaMemcpyDeviceToHost, st) !=
        cudaSuccess)
        return HIGGS_ERR_CUDA;
    return HIGGS_OK;
}

int higgs_linear_host_batch(int32_t count, const higgs_desc* const* descs, const void* const* x_hosts, int64_t B,
                            const void* const* packed, const void* const* scales, const float* const* grids,
                            void* const* y_hosts, int y_dtype, void* const* workspaces,
                            const size_t* workspace_bytes, void* stream) {
    if (count < 0) return HIGGS_ERR_INVALID_ARG;
    if (count == 0) return HIGGS_OK;
    if (!descs || !x_hosts || !packed || !scales || !grids || !y_hosts || !workspaces || !workspace_bytes)
        return HIGGS_ERR_INVALID_ARG;
    if (y_dtype != HIGGS_F32 && y_dtype != HIGGS_BF16) return HIGGS_ERR_UNSUPPORTED;
    if (B < 0) return HIGGS_ERR_INVALID_ARG;
    cudaStream_t st = as_stream(stream);
    for (int i = 0; i < count; ++i) {
        const higgs_desc* d = descs[i];
        int rc = check_desc(d);
        if (rc != HIGGS_OK) return rc;
        if (B == 0 || d->N == 0) continue;
        if (!x_hosts[i] || !y_hosts[i] || !workspaces[i] || !aligned(workspaces[i], 256)) return HIGGS_ERR_INVALID_ARG;
        const size_t inner = higgs_workspace_bytes(d, HIGGS_OP_LINEAR, B);
        const size_t xb = align_up((size_t)B * d->K * 2, 256);
        const size_t ybytes = (size_t)B * d->N * (y_dtype == HIGGS_F32 ? 4 : 2);
        if (workspace_bytes[i] < inner + xb + align_up(ybytes, 256)) return HIGGS_ERR_WORKSPACE;
        uint8_t* ws = static_cast<uint8_t*>(workspaces[i]);
        const void* x_dev = nullptr;
        for (int j = 0; j < i && !x_dev; ++j) {       // an earlier layer staged the same activations
            if (x_hosts[j] == x_hosts[i] && descs[j]->K == d->K && descs[j]->N != 0)
                x_dev = static_cast<const uint8_t*>(workspaces[j]) + higgs_workspace_bytes(descs[j], HIGGS_OP_LINEAR, B);
        }
        if (!x_dev) {
            if (cudaMemcpyAsync(ws + inner, x_hosts[i], (size_t)B * d->K * 2, cudaMemcpyHostToDevice, st) != cudaSuccess)
                return HIGGS_ERR_CUDA;
            x_dev = ws + inner;
        }
        void* y_dev = ws + inner + xb;
        rc = higgs_linear(d, x_dev, B, packed[i], scales[i], grids[i], y_dev, y_dtype, ws, inner, stream);
        if (rc != HIGGS_OK) return rc;
        if (cudaMemcpyAsync(y_hosts[i], y_dev, ybytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return HIGGS_ERR_CUDA;
    }
    return HIGGS_OK;
}

// ---- one host block in, one host block out ---------------------------------------------------------------------
static size_t host_block_inner(int32_t count, const higgs_desc* const* descs, int64_t B) {
    // the products run one after the other on the stream and share one inner workspace: the largest any of them -
    // or any run of up to four layers taken together by higgs_linear_multi - needs
    size_t inner = 0;
    for (int i = 0; i < count; ++i) {
        for (int n = 1; n <= kMaxMulti && i + n <= count; ++n) {
            const size_t w = n == 1 ? higgs_workspace_bytes(descs[i], HIGGS_OP_LINEAR, B)
                                    : higgs_linear_multi_workspace_bytes(n, descs + i, B);
            inner = w > inner ? w : inner;
        }
    }
    return align_up(inner, 256);
}

size_t higgs_linear_host_block_workspace_bytes(int32_t count, const higgs_desc* const* descs, int64_t B, size_t x_block_bytes,
                                               size_t y_block_bytes) {
    if (count < 1 || !descs || B < 1) return 0;
    for (int i = 0; i < count; ++i)
        if (check_desc(descs[i]) != HIGGS_OK) return 0;
    return host_block_inner(count, descs, B) + align_up(x_block_bytes, 256) + align_up(y_block_bytes, 256);
}

int higgs_linear_host_block(int32_t count, const higgs_desc* const* descs, const void* x_host_block, size_t x_block_bytes,
                            const size_t* x_offsets, int64_t B, const void* const* packed, const void* const* scales,
                            const float* const* grids, void* y_host_block, size_t y_block_bytes, const size_t* y_offsets,
                            int y_dtype, void* workspace, size_t workspace_bytes, void* stream) {
    if (count < 0) return HIGGS_ERR_INVALID_ARG;
    if (count == 0) return HIGGS_OK;
    if (!descs || !x_offsets || !y_offsets || !packed || !scales || !grids) return HIGGS_ERR_INVALID_ARG;
    if (y_dtype != HIGGS_F32 && y_dtype != HIGGS_BF16) return HIGGS_ERR_UNSUPPORTED;
    if (B < 0) return HIGGS_ERR_INVALID_ARG;
    const size_t esz = y_dtype == HIGGS_F32 ? 4 : 2;
    for (int i = 0; i < count; ++i) {
        const int rc = check_desc(descs[i]);
        if (rc != HIGGS_OK) return rc;
        if (x_offsets[i] % 16 || y_offsets[i] % 16) return HIGGS_ERR_INVALID_ARG;
        if (x_offsets[i] + (size_t)B * descs[i]->K * 2 > x_block_bytes) return HIGGS_ERR_INVALID_ARG;
        if (y_offsets[i] + (size_t)B * descs[i]->N * esz > y_block_bytes) return HIGGS_ERR_INVALID_ARG;
    }
    if (B == 0) return HIGGS_OK;
    if (!x_host_block || !y_host_block || !workspace || !aligned(workspace, 256)) return HIGGS_ERR_INVALID_ARG;
    if (workspace_bytes < higgs_linear_host_block_workspace_bytes(count, descs, B, x_block_bytes, y_block_bytes)) return HIGGS_ERR_WORKSPACE;
    const size_t inner = host_block_inner(count, descs, B);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    uint8_t* x_dev = ws + inner;
    uint8_t* y_dev = x_dev + align_up(x_block_bytes, 256);
    cudaStream_t st = as_stream(stream);
    if (cudaMemcpyAsync(x_dev, x_host_block, x_block_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return HIGGS_ERR_CUDA;
    for (int i = 0; i < count;) {
        // consecutive layers with the same input, grid table, grid, group size, K and seed run as one product
        int n = 1;
        while (i + n < count && n < kMaxMulti && x_offsets[i + n] == x_offsets[i] && grids[i + n] == grids[i] &&
               descs[i + n]->p == descs[i]->p && descs[i + n]->n == descs[i]->n && descs[i + n]->K == descs[i]->K &&
               descs[i + n]->rht_seed == descs[i]->rht_seed)
            ++n;
        int rc;
        if (n == 1) {
            rc = descs[i]->N == 0 ? HIGGS_OK
                                  : higgs_linear(descs[i], x_dev + x_offsets[i], B, packed[i], scales[i], grids[i], y_dev + y_offsets[i],
                                                 y_dtype, ws, inner, stream);
        } else {
            void* ys[kMaxMulti];
            for (int j = 0; j < n; ++j) ys[j] = y_dev + y_offsets[i + j];
            rc = higgs_linear_multi(n, descs + i, x_dev + x_offsets[i], B, packed + i, scales + i, grids[i], ys, y_dtype, ws, inner,
                                    stream);
        }
        if (rc != HIGGS_OK) return rc;
        i += n;
    }
    if (cudaMemcpyAsync(y_host_block, y_dev, y_block_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return HIGGS_ERR_CUDA;
    return HIGGS_OK;
}

size_t higgs_linear_host_workspace_bytes(const higgs_desc* d, int64_t B, int y_dtype) {
    const size_t inner = higgs_workspace_bytes(d, HIGGS_OP_LINEAR, B);
    if (inner == 0) return 0;
    return inner + align_up((size_t)B * d->K * 2, 256) + align_up((size_t)B * d->N * (y_dtype == HIGGS_F32 ? 4 : 2), 256);
}

size_t higgs_rotated_bytes(const higgs_desc* d, int64_t B) {
    if (check_desc(d) != HIGGS_OK || B < 1) return 0;
    return tc_eligible(*d, B) ? tc_workspace_bytes(*d, B) : (size_t)B * d->K * 2;
}

int higgs_rotated_layout(const higgs_desc* d, int64_t B) {
    if (check_desc(d) != HIGGS_OK || B < 1) return -1;
    return tc_eligible(*d, B) ? tc_batch_tile(B) : 0;
}

int higgs_linear_k_splits(const higgs_desc* d, int64_t B) {
    if (check_desc(d) != HIGGS_OK || B < 1 || d->N == 0 || d->K == 0) return 0;
    if (tc_eligible(*d, B)) return tc_k_split(*d, B);
    return linear_k_chunks(*d, B);
}

int higgs_linear_uses_atomics(const higgs_desc* d, int64_t B) {
    if (check_desc(d) != HIGGS_OK || B < 1 || d->N == 0 || d->K == 0) return 0;
    if (tc_eligible(*d, B)) return 0;
    return linear_uses_atomics(*d, B) ? 1 : 0;
}

int higgs_linear_launch_count(const higgs_desc* d, int64_t B, int y_dtype) {
    if (check_desc(d) != HIGGS_OK || B < 1 || d->N == 0) return 0;
    if (tc_eligible(*d, B)) return 2;
    if (linear_fused_eligible(*d, B)) return 1;
    const bool split = linear_uses_atomics(*d, B);
    return 1 + (int)((B + 15) / 16) + ((split && y_dtype == HIGGS_BF16) ? 1 : 0);
}

int higgs_device_status(void* stream, int clear) { return read_device_status(as_stream(stream), clear); }

int higgs_rht(const higgs_desc* d, const void* x, int x_dtype, int64_t rows, float* out, int normalised, void* stream) {
    int rc = check_desc(d);
    if (rc != HIGGS_OK) return rc;
    if (rows < 0) return HIGGS_ERR_INVALID_ARG;
    if (rows == 0 || d->K == 0) return HIGGS_OK;
    if (!x || !out || !aligned(x, 16) || !aligned(out, 16)) return HIGGS_ERR_INVALID_ARG;
    return launch_rht_debug(*d, x, x_dtype, rows, out, normalised, as_stream(stream));
}

int higgs_pack_codes(const higgs_desc* d, const uint8_t* canonical, void* packed_out, void* stream) {
    int rc = check_desc(d);
    if (rc != HIGGS_OK) return rc;
    if (d->N == 0 || d->K == 0) return HIGGS_OK;
    if (!canonical || !packed_out || !aligned(packed_out, 16) || !aligned(canonical, 16)) return HIGGS_ERR_INVALID_ARG;
    rc = launch_pack(*d, canonical, packed_out, as_stream(stream));
    return rc != HIGGS_OK ? rc : launch_stream_fence(as_stream(stream));
}

int higgs_unpack_codes(const higgs_desc* d, const void* packed, uint8_t* canonical_out, void* stream) {
    int rc = check_desc(d);
    if (rc != HIGGS_OK) return rc;
    if (d->N == 0 || d->K == 0) return HIGGS_OK;
    if (!packed || !canonical_out || !aligned(packed, 16)) return HIGGS_ERR_INVALID_ARG;
    return launch_unpack(*d, packed, canonical_out, as_stream(stream));
}

}  // extern "C"
