/*
 * higgs.h - C ABI of the B200 (sm_100a) HIGGS quantized linear layer.
 *
 * The library implements the data-parallel hot path of HIGGS ("Hadamard
 * Incoherence and Gaussian MSE-optimal GridS"): the encoder of Algorithm 1
 * (RHT-VQ) with the grid of Algorithm 2, and the rotated-space product of
 * Appendix F ("Rotating Activations") with the lookup-table dequantisation
 * discussed in Section 4.3.
 *
 * Symbols: N = output features (rows of W), K = input features, B = tokens,
 * g = scale / rotation group size along K, p = grid dimension, n = grid size,
 * xi = RHT seed.  W is [N][K] row-major; groups are W[r, i*g:(i+1)*g]
 * (Appendix F).  Codes are 0-based (Algorithm 1 prints them 1-based).
 *
 * Conventions for every entry point
 *   - Pointers marked "device" are caller-allocated device memory; the library
 *     never allocates, frees, retains or reallocates them.  Pointers marked
 *     "host" are ordinary host memory.
 *   - All device work is enqueued on the caller's stream (a cudaStream_t passed
 *     as void*; NULL = the legacy default stream).  No call synchronises.
 *   - The return value is a higgs_status; HIGGS_OK means the work was enqueued.
 *     Nothing is enqueued when another value is returned.
 *   - Inputs must be finite; this is a precondition, not checked on the device.
 *   - There is no CPU fallback: without a CUDA device every compute call
 *     returns HIGGS_ERR_CUDA.
 *
 * The sign function of the randomised Hadamard transform (part of the ABI):
 *   out(xi, m):  z = xi + (m+1) * 0x9E3779B97F4A7C15            (mod 2^64)
 *                z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9
 *                z = (z ^ (z >> 27)) * 0x94D049BB133111EB
 *                z =  z ^ (z >> 31)
 *   i.e. output number m of the splitmix64 stream seeded with xi, and
 *   sign(xi, j) = -1 if bit (j mod 64) of out(xi, floor(j / 64)) is set, else +1.
 * One sign per input index j in [0, K), shared by every row of W and every
 * token, so that the activations are rotated once (Appendix F, "Rotating
 * Activations": activations and weights are transformed with one seed over
 * identical groups).
 *
 * The transform itself: RHT(v) = H * diag(sign) * v on each group of g values,
 * H the Sylvester-ordered Hadamard matrix H[i][j] = (-1)^popcount(i & j).
 * The encoder uses H unnormalised (Algorithm 1: entries of the rotated unit
 * vector are approximately N(0,1)); the activations use H / sqrt(g), which is
 * orthonormal, i.e. a random rotation (Appendix F).
 *
 * Ordering of producers and consumers on a stream.  The product kernels are
 * launched so that they may begin (table build, first weight copies) before
 * the previous kernel of the stream has finished; they wait for it before
 * they touch x, y or the workspace.  packed, scales and grid are therefore
 * read early: they must not be written by work that is still running when a
 * higgs_linear* call is enqueued behind it.  The library's own producers
 * (higgs_quantize, higgs_pack_codes, higgs_make_grid*, higgs_make_uniform_grid)
 * end with a kernel that is launched without that early-start permission, so
 * calling them and a product back to back on one stream is safe; a caller
 * who fills these buffers with kernels of their own must leave one ordinary
 * kernel launch or event between those kernels and the product.
 */
#ifndef HIGGS_H_
#define HIGGS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum higgs_status {
    HIGGS_OK = 0,
    HIGGS_ERR_INVALID_ARG = 1,   /* null pointer, negative size, misaligned pointer            */
    HIGGS_ERR_UNSUPPORTED = 2,   /* (p, n, g, dtype, shape) combination has no kernel          */
    HIGGS_ERR_WORKSPACE = 3,     /* workspace smaller than higgs_workspace_bytes() asks        */
    HIGGS_ERR_CUDA = 4,          /* a CUDA runtime call failed (no device, launch error)        */
    HIGGS_ERR_TIMEOUT = 5,       /* a bounded device-side wait ran out (read from a status word) */
    HIGGS_ERR_STATIC_SCRATCH = 6 /* request does not fit the library's built-in scratch array       */
} higgs_status;

typedef enum higgs_dtype { HIGGS_F32 = 0, HIGGS_F16 = 1, HIGGS_BF16 = 2 } higgs_dtype;

typedef enum higgs_op { HIGGS_OP_QUANTIZE = 0, HIGGS_OP_LINEAR = 1, HIGGS_OP_MAKE_GRID = 2, HIGGS_OP_MAKE_GRID_SEEDED = 3 } higgs_op;

/* Version of the packed code stream and scale layouts this library writes and reads (higgs_desc.layout_version). */
#define HIGGS_LAYOUT_VERSION 1

/*
 * Description of one quantized matrix.  Supported: g = 1024; (p, n) in
 * {(2,256), (2,64), (2,16), (1,16), (1,8), (1,4), (1,256)} - the 4-, 3- and 2-bit
 * vector and scalar grids and the 8-bit scalar one; N a multiple of 16, K a multiple of g.
 * Anything else returns HIGGS_ERR_UNSUPPORTED (never padded silently).
 * scale_dtype must be HIGGS_F16: one 16-bit scale per (row, group), which is
 * what the paper's bit counts imply (4.02 = 4 + 16/1024 in the appendix on
 * experiment configurations).  layout_version must be HIGGS_LAYOUT_VERSION: packed
 * buffers are only meaningful to the library version that wrote them, and a
 * descriptor saved beside them says which that was.
 */
typedef struct higgs_desc {
    int32_t p;
    int32_t n;
    int32_t g;
    int32_t scale_dtype;
    uint64_t rht_seed; /* xi */
    int64_t N;
    int64_t K;
    int32_t layout_version; /* HIGGS_LAYOUT_VERSION */
    int32_t reserved;       /* 0 */
} higgs_desc;

/* Text for a status code (static storage, never NULL). */
const char* higgs_status_string(int status);

/* Host evaluation of the ABI's sign function: returns +1 or -1. */
int higgs_sign(uint64_t rht_seed, int64_t j);

/* Bytes of the packed code stream (kernel-native, opaque layout; log2(n)/p
 * bits per weight), of the scale array (N * K/g values of scale_dtype), and of the
 * canonical code array ([N][K/p], one byte per code).  0 if unsupported.   */
size_t higgs_packed_bytes(const higgs_desc* desc);
size_t higgs_scales_bytes(const higgs_desc* desc);
size_t higgs_canonical_bytes(const higgs_desc* desc);

/* Scratch bytes the given operation needs for batch B (B ignored unless
 * op == HIGGS_OP_LINEAR; for HIGGS_OP_MAKE_GRID and HIGGS_OP_MAKE_GRID_SEEDED
 * desc->K holds the number of samples and desc->p, desc->n the grid; the other
 * descriptor fields are ignored for these two).  Workspaces must be 256-byte
 * aligned.  Contents need not be initialised and are undefined afterwards.  */
size_t higgs_workspace_bytes(const higgs_desc* desc, int op, int64_t B);

/*
 * Section 4.3, "Constrained HIGGS": the uniform n-level scalar grid, symmetric about zero, whose step minimises
 * the expected squared error of rounding N(0,1) (closed-form MSE, golden-section search in fp64 on the device).
 * With n = 256 this is the paper's 8-bit option ("CH8"); use it with p = 1.
 *   grid_out   device, [n] fp32 (= [n][1])
 *   step_out   device, optional: the step
 *   mse_out    device, optional: the expected squared error per weight
 * 2 <= n <= 256, else HIGGS_ERR_UNSUPPORTED.  Asynchronous on `stream`.
 */
int higgs_make_uniform_grid(int n, float* grid_out, float* step_out, float* mse_out, void* stream);

/*
 * Algorithm 2, first line: the Gaussian-MSE-optimal grid.  The paper names the
 * procedure (CLVQ) without its parameters; this library runs the batch (Lloyd)
 * fixed-point iteration on the caller's samples of N(0, I_p): centres start at
 * the first n samples; every iteration assigns each sample to its nearest
 * centre (ties to the lowest index) and moves each centre to the mean of its
 * samples (an empty cell keeps its centre); it stops when no assignment
 * changes or after max_iters iterations; centres are then sorted
 * lexicographically.
 *   samples      device, [num_samples][p] fp32, num_samples >= n
 *   grid_out     device, [n][p] fp32
 *   mse_out      device, optional: per-dimension MSE of the final assignment on
 *                the samples
 *   iters_out    device, optional: iterations run (int32), negative if
 *                max_iters was reached without convergence
 * Distances are fp32, sums fp64; the result is a fixed point of the same
 * iteration the fp64 definition runs but need not be bit-identical to it.
 * 1 <= p <= 4 and 1 <= n <= 4096 (n need not be a power of two), else
 * HIGGS_ERR_UNSUPPORTED.
 */
int higgs_make_grid(int p, int n, const float* samples, int64_t num_samples, int max_iters,
                    float* grid_out, float* mse_out, int32_t* iters_out,
                    void* workspace, size_t workspace_bytes, void* stream);

/*
 * Algorithm 2's grid with the samples drawn by the library: 2^log2_samples points of N(0, I_p) from sample_seed, then
 * the iteration of higgs_make_grid on them.  Sample i, coordinate k is sqrt(-2 ln u1) cos(2 pi u2) with
 * u1 = (bits 40..63 of z + 0.5) / 2^24, u2 = (bits 16..39 of z + 0.5) / 2^24, z = out(sample_seed, i p + k) of the
 * splitmix64 stream defined above (fp32 arithmetic).  workspace: higgs_workspace_bytes(desc, HIGGS_OP_MAKE_GRID_SEEDED,
 * 0) bytes with desc->K = 2^log2_samples (it holds the samples too).  1 <= log2_samples <= 24.  Other arguments and
 * errors as higgs_make_grid.  higgs_gaussian_samples writes the same samples ([num_samples][p] fp32, device) alone.
 */
int higgs_make_grid_seeded(int p, int n, uint64_t sample_seed, int log2_samples, int max_iters,
                           float* grid_out, float* mse_out, int32_t* iters_out,
                           void* workspace, size_t workspace_bytes, void* stream);
int higgs_gaussian_samples(int p, uint64_t sample_seed, int64_t num_samples, float* samples_out, void* stream);

/*
 * Algorithm 1 (RHT-VQ) on every row of W.  Per (row r, group i):
 *   s = ||w||_2;  w+ = H diag(sign) (w / s);  code_t = nearest grid point of
 *   the t-th consecutive p-tuple of w+ (exhaustive search, fp32 squared
 *   distances, lowest index on exact ties);  stored scale = s / sqrt(g).
 * A group of zeros gets scale 0 and the code of the point nearest the origin.
 *   W              device, [N][K] row-major, w_dtype in {HIGGS_F32, HIGGS_BF16}
 *   grid           device, [n][p] fp32
 *   packed_out     device, higgs_packed_bytes() bytes, 16-byte aligned
 *   scales_out     device, higgs_scales_bytes() bytes, 16-byte aligned: fp16 scales stored
 *                  tile-major, element (r, i) at index ((r / 16) * (K/g) + i) * 16 + r % 16
 *   canonical_out  device, optional, [N][K/p] one byte per code (for checking), 16-byte aligned
 *   workspace      device, 256-byte aligned, higgs_workspace_bytes(desc, HIGGS_OP_QUANTIZE, 0) bytes: required when
 *                  canonical_out is NULL (HIGGS_ERR_INVALID_ARG / HIGGS_ERR_WORKSPACE otherwise); optional with
 *                  canonical_out (without it a large layer's packed stream is written by a second kernel)
 */
int higgs_quantize(const higgs_desc* desc, const void* W, int w_dtype, const float* grid,
                   void* packed_out, void* scales_out, uint8_t* canonical_out,
                   void* workspace, size_t workspace_bytes, void* stream);

/* The search table of the encoder, built once per grid.  Layers of at least 2 M weights are encoded with an exact
 * pruned nearest-point search (same codes as the exhaustive scan of Algorithm 1's rounding step, bit for bit) over a
 * table of candidate lists that depends on the grid only; higgs_quantize builds it on every call (in its workspace),
 * higgs_quantize_prepared takes one built beforehand - worthwhile when many layers share a grid, as the layers of a
 * model do.  The paper does not describe the search; this is an implementation device with no counterpart there.
 *   higgs_encoder_table_bytes  size of the table for (p, n); 0 if the pair has no kernel
 *   higgs_make_encoder_table   grid: device [n][p] fp32; table_out: device, 16-byte aligned; asynchronous on `stream`
 *   higgs_quantize_prepared    as higgs_quantize; table: device, from higgs_make_encoder_table for the same (p, n) and
 *                              grid values, or NULL (then identical to higgs_quantize)                              */
size_t higgs_encoder_table_bytes(int p, int n);
int higgs_make_encoder_table(int p, int n, const float* grid, void* table_out, void* stream);
int higgs_quantize_prepared(const higgs_desc* desc, const void* W, int w_dtype, const float* grid, const void* table,
                            void* packed_out, void* scales_out, uint8_t* canonical_out,
                            void* workspace, size_t workspace_bytes, void* stream);

/*
 * Appendix F, "Rotating Activations": y = x W^T computed in the rotated space.
 *   x+ = (H / sqrt(g)) diag(sign) x per token and K-group (same xi as the
 *   encoder);  y[b][r] = sum_i scale[r][i] * sum_t < G[code[r][i][t]], x+[b][i][tp:(t+1)p] >.
 * Grid entries and x+ are rounded to fp16 for the tensor-core operands;
 * products are exact and accumulation is fp32; scales are applied in fp32.
 *   x        device, [B][K] row-major bf16, B >= 1
 *   packed   device, from higgs_quantize / higgs_pack_codes
 *   scales   device, tile-major fp16 scales as written by higgs_quantize
 *   grid     device, [n][p] fp32
 *   y        device, [B][N] row-major, y_dtype in {HIGGS_F32, HIGGS_BF16}
 * Kernels behind the call: for one or two tokens (K up to 8192) a single kernel
 * that rotates the activations in its prologue; up to 16 tokens a rotation
 * kernel and the small-batch product kernel; above that (and from 9 tokens
 * for layers with at least 4096 rows, 4096 inputs and 16 M weights) a rotation kernel and the tcgen05 kernel.
 * When the small-batch kernel splits K over more than two thread blocks the
 * partial sums meet in fp32 atomics, so the last bits of y may differ from run
 * to run (higgs_linear_uses_atomics); every other path is bit-reproducible.  The one-call form and the two-call
 * form below agree to fp16 rounding of x+ (the fused prologue orders the
 * butterflies differently), not bit for bit.
 */
int higgs_linear(const higgs_desc* desc, const void* x, int64_t B,
                 const void* packed, const void* scales, const float* grid,
                 void* y, int y_dtype,
                 void* workspace, size_t workspace_bytes, void* stream);

/*
 * The two halves of higgs_linear as separate calls (Section 4.3 observes that
 * the Hadamard transform does not have to be part of the matrix product).
 *   higgs_rotate_activations: x (device [B][K] bf16) -> xdag_out (device,
 *     higgs_rotated_bytes(desc, B) bytes of fp16) = (H / sqrt(g)) diag(sign) x
 *     per K-group.  The storage order is internal to the library and named by
 *     higgs_rotated_layout(desc, B): 0 = [B][K] with the 32 input pairs of every
 *     64-input block in the product kernel's fragment order (B <= 16, or layers
 *     the tensor-core path does not take), t > 0 = blocked operand tiles of t
 *     tokens for the tensor-core path.
 *   higgs_linear_prerotated: the product of Appendix F on already rotated
 *     activations; other arguments as higgs_linear.  xdag may be shared by
 *     layers with the same K, seed and higgs_rotated_layout (e.g. q, k, v).
 * higgs_linear(x) computes what higgs_linear_prerotated(higgs_rotate_activations(x)) does.
 */
int higgs_rotate_activations(const higgs_desc* desc, const void* x, int64_t B, void* xdag_out, void* stream);
size_t higgs_rotated_bytes(const higgs_desc* desc, int64_t B);
int higgs_rotated_layout(const higgs_desc* desc, int64_t B);
int higgs_linear_prerotated(const higgs_desc* desc, const void* xdag, int64_t B,
                            const void* packed, const void* scales, const float* grid,
                            void* y, int y_dtype,
                            void* workspace, size_t workspace_bytes, void* stream);

/*
 * higgs_linear that also leaves the rotated activations behind, for the first of several layers that read the same
 * x (q before k and v; gate before up) - Section 4.3 notes that the transform of the activations can be isolated from
 * the product of Appendix F, so layers with a common input need it once: y as higgs_linear, and xdag_out (device, higgs_rotated_bytes(desc, B) bytes,
 * 16-byte aligned) receives what higgs_rotate_activations(desc, x, B) writes, to be passed to
 * higgs_linear_prerotated for the other layers (same K, seed and higgs_rotated_layout).  For one or two tokens on a
 * layer whose K is not split this is ONE launch - the product kernel rotates x itself and one of its blocks stores
 * the result - instead of a rotation launch followed by a product launch; otherwise it is those two launches.
 * xdag_out is complete when the call's last kernel has completed (stream order).
 */
int higgs_linear_share(const higgs_desc* desc, const void* x, int64_t B, const void* packed, const void* scales,
                       const float* grid, void* y, int y_dtype, void* xdag_out, void* workspace,
                       size_t workspace_bytes, void* stream);

/*
 * Several layers that read the same activations (q, k, v; gate, up) as ONE product: Appendix F's product is
 * independent per output row, so matrices with the same K, grid, group size and seed are one layer over their
 * concatenated rows - the activations are rotated once and, for batches up to 16 (the small-batch kernel, K ranges
 * not meeting in atomics), one kernel launch per 16 tokens streams all of them; for one or two tokens that launch also
 * does the rotation.  Other shapes and batches run as one higgs_linear per matrix (same results, no gain).
 *   count <= 4; descs[i], packed[i], scales[i], ys[i] (device [B][descs[i]->N] of y_dtype) belong to matrix i;
 *   descs must agree in p, n, g, K, rht_seed (else HIGGS_ERR_INVALID_ARG); grid and x are common;
 *   workspace: higgs_linear_multi_workspace_bytes(count, descs, B) bytes.  The arrays are HOST arrays.
 * Results equal those of higgs_linear on each matrix (bit for bit where neither uses atomics).
 * higgs_linear_multi_launch_count: kernels the call enqueues.
 */
int higgs_linear_multi(int32_t count, const higgs_desc* const* descs, const void* x, int64_t B,
                       const void* const* packed, const void* const* scales, const float* grid,
                       void* const* ys, int y_dtype, void* workspace, size_t workspace_bytes, void* stream);
size_t higgs_linear_multi_workspace_bytes(int32_t count, const higgs_desc* const* descs, int64_t B);
int higgs_linear_multi_launch_count(int32_t count, const higgs_desc* const* descs, int64_t B, int y_dtype);

/*
 * Row-sharded layer with the all-gather fused into the product's epilogue (Appendix F's product is independent per
 * output row, and the rotation is local to a 1024-group of inputs, so a layer splits over devices by rows with no
 * exchange of weights): this device holds rows [row_offset, row_offset + desc->N) of a layer with `ld` rows in all
 * (desc, packed, scales describe the SHARD), every device holds the full activations x, and the shard's outputs are
 * written straight into columns [row_offset, row_offset + desc->N) of EVERY destination
 *   y_dsts[i] : device-accessible [B][ld] of y_dtype, i < n_dst <= 8 - this device's own output buffer first, then the
 *               peer-mapped pointers of the other devices' buffers (cudaDeviceEnablePeerAccess / IPC / symmetric
 *               memory; plain stores over NVLink, one per destination).
 * The kernels store to all destinations from their epilogue (a K-split small-batch product sums into the workspace
 * first and a copy kernel spreads the result).  The call neither waits for nor signals other devices: the caller
 * orders "all shards written" before any reader (e.g. a barrier on the participating streams), and no two shards
 * overlap in columns.  row_offset a multiple of 16, ld a multiple of 8, ld >= row_offset + desc->N; y_dsts is a HOST
 * array.  Other arguments, errors and workspace as higgs_linear.
 */
int higgs_linear_gather(const higgs_desc* desc, const void* x, int64_t B, const void* packed, const void* scales,
                        const float* grid, void* const* y_dsts, int32_t n_dst, int64_t ld, int64_t row_offset,
                        int y_dtype, void* workspace, size_t workspace_bytes, void* stream);

/*
 * The row range of a layer with N rows that rank `rank` of `world` devices holds when the layer is sharded by rows
 * for higgs_linear_gather (rows are independent in Algorithm 1 and in Appendix F's product): contiguous ranges of
 * whole units of `multiple` rows (a multiple of 16; 128 keeps every shard on the tensor-core path), the remainder
 * units going to the first ranks.  HOST function.  *begin_out = first row, *count_out = rows of the shard.
 * HIGGS_ERR_UNSUPPORTED if N is not a multiple of `multiple`.
 */
int higgs_shard_rows(int64_t N, int32_t world, int32_t rank, int32_t multiple, int64_t* begin_out, int64_t* count_out);

/*
 * Layer sharded along K on group boundaries (Appendix F: the rotation acts inside a 1024-group, so a device that holds
 * inputs [k0, k0 + K_r) of every row, k0 a multiple of 1024, can rotate its slice of x and multiply it on its own; the
 * fp32 partial outputs of the devices are then summed).  A K-shard is an ordinary layer of K_r inputs whose sign
 * sequence starts at input k0: higgs_shard_seed(xi, k0) is the seed that makes sign(seed', j) = sign(xi, k0 + j), so
 * a shard encoded and multiplied with {N, K_r, seed'} carries exactly the codes and signs of columns [k0, k0 + K_r)
 * of the unsharded layer.  (HOST function.)
 *
 * higgs_linear_kshard: this device's partial product, written from the kernels' epilogues (plain stores, own
 * memory and peer-mapped memory alike, one store per destination) into slot `rank` of EVERY device's slot buffer
 *   slot_bufs[i] : device-accessible fp32 [world][B][N] of device i (i = rank: this device's own), a HOST array;
 * desc/x_shard/packed/scales describe the shard (x_shard is [B][K_r] bf16).  It neither waits for nor signals other
 * devices: the caller orders "all partials written" before higgs_reduce_slots (a barrier of the process group).
 * higgs_reduce_slots: y[i] = slots[0][i] + slots[1][i] + ... in slot order (bit-reproducible), count = B * N values
 * (a multiple of 4), y fp32 or bf16.  Both asynchronous on `stream`; errors and workspace as higgs_linear_gather.
 */
uint64_t higgs_shard_seed(uint64_t rht_seed, int64_t k_offset);
int higgs_linear_kshard(const higgs_desc* desc, const void* x_shard, int64_t B, const void* packed, const void* scales,
                        const float* grid, void* const* slot_bufs, int32_t world, int32_t rank,
                        void* workspace, size_t workspace_bytes, void* stream);
int higgs_reduce_slots(const float* slots, int32_t world, int64_t count, void* y, int y_dtype, void* stream);

/*
 * higgs_linear with HOST activations and HOST output (Appendix F product; the
 * weights stay resident on the device): copies x_host ([B][K] bf16, ideally
 * pinned) to the device, runs higgs_linear, copies y ([B][N] of y_dtype) back to
 * y_host, all enqueued on `stream`; the caller synchronises the stream before
 * reading y_host.  workspace is DEVICE memory of at least
 * higgs_linear_host_workspace_bytes() bytes (it also stages x and y).
 */
int higgs_linear_host(const higgs_desc* desc, const void* x_host, int64_t B,
                      const void* packed, const void* scales, const float* grid,
                      void* y_host, int y_dtype,
                      void* workspace, size_t workspace_bytes, void* stream);
size_t higgs_linear_host_workspace_bytes(const higgs_desc* desc, int64_t B, int y_dtype);

/*
 * `count` higgs_linear_host calls (each the rotated-space product of Appendix F from host activations to a host
 * output) enqueued by ONE call - the products of a transformer block, say - so that the
 * host spends one library call, not `count`, per step.  Argument i of every array belongs to layer i
 * (descs[i], x_hosts[i], packed[i], scales[i], grids[i], y_hosts[i], workspaces[i], workspace_bytes[i]); B and
 * y_dtype are common.  Layers that name the SAME x_hosts pointer and have the same K (q/k/v; gate/up) share one
 * host-to-device copy: the later layer reads the staged copy in the earlier layer's workspace, so those workspaces
 * must stay untouched until the stream has passed this call.  Returns the first error and enqueues nothing further
 * after it.  Asynchronous on `stream`; the caller synchronises before reading any y_hosts[i].
 */
int higgs_linear_host_batch(int32_t count, const higgs_desc* const* descs, const void* const* x_hosts, int64_t B,
                            const void* const* packed, const void* const* scales, const float* const* grids,
                            void* const* y_hosts, int y_dtype, void* const* workspaces,
                            const size_t* workspace_bytes, void* stream);

/*
 * The same with ONE host block in and ONE host block out, so that a step costs two copies whatever the number of
 * layers: x_host_block (ideally pinned) holds every distinct input of the step, layer i reads [B][K_i] bf16 at byte
 * offset x_offsets[i] (layers with a common input name the same offset); y_host_block receives layer i's [B][N_i]
 * output of y_dtype at byte offset y_offsets[i] (offsets multiples of 16, ranges inside the blocks, else
 * HIGGS_ERR_INVALID_ARG).  Enqueued on `stream`: one host-to-device copy of the input block, the products of Appendix F
 * in order - consecutive layers that name the same input offset, grid table, (p, n), K and seed run as one product
 * (higgs_linear_multi) - and one device-to-host copy of the output block.  workspace: ONE device buffer of
 * higgs_linear_host_block_workspace_bytes() bytes (inner scratch shared by the products, which run one after the
 * other, plus the two staged blocks).  The caller synchronises before reading y_host_block.  Arrays are HOST arrays.
 */
int higgs_linear_host_block(int32_t count, const higgs_desc* const* descs, const void* x_host_block, size_t x_block_bytes,
                            const size_t* x_offsets, int64_t B, const void* const* packed, const void* const* scales,
                            const float* const* grids, void* y_host_block, size_t y_block_bytes, const size_t* y_offsets,
                            int y_dtype, void* workspace, size_t workspace_bytes, void* stream);
size_t higgs_linear_host_block_workspace_bytes(int32_t count, const higgs_desc* const* descs, int64_t B,
                                               size_t x_block_bytes, size_t y_block_bytes);

/*
 * higgs_linear without a workspace argument, for callers that cannot allocate
 * device memory (code running where cudaMalloc is off limits, plugins that are
 * only handed their input and output buffers, processes whose memory pool
 * belongs to another component).  The paper has no counterpart: this is purely
 * an interface convenience.  The result is the same as higgs_linear's.
 *
 * The scratch lives in one fixed array of higgs_linear_static_capacity() bytes
 * (4 MiB) inside the library image; every GPU that loads the library holds it
 * until the process exits.  A call whose higgs_workspace_bytes(desc,
 * HIGGS_OP_LINEAR, B) exceeds that capacity returns HIGGS_ERR_STATIC_SCRATCH and
 * enqueues nothing; 4 MiB covers every Llama-shaped layer up to 28672 x 8192
 * at B <= 16.
 *
 * The call allocates nothing and calls no allocating routine.  Its first call on
 * a device looks the array's address up (once per device, with that device
 * current); make that first call before starting any stream capture.  All calls
 * on a device share the one array: it keeps whatever the previous call left, the
 * kernels overwrite or clear everything they read, and two calls that overlap on
 * the GPU (different streams, or the same shape replayed concurrently) race on
 * it - serialise them.  x, packed, scales, grid and y are caller-owned device
 * buffers exactly as for higgs_linear.
 */
int higgs_linear_static(const higgs_desc* desc, const void* x, int64_t B,
                        const void* packed, const void* scales, const float* grid,
                        void* y, int y_dtype, void* stream);
size_t higgs_linear_static_capacity(void);

/*
 * Every device-side wait in this library is bounded.  If one runs out, the kernel
 * gives up, and the library's device status word becomes HIGGS_ERR_TIMEOUT.
 * This call synchronises `stream`, returns the word (HIGGS_OK if no wait ever
 * ran out) and, if clear != 0, resets it.  Results computed by a launch that
 * timed out are undefined.
 */
int higgs_device_status(void* stream, int clear);

/*
 * Measurement and self-check helpers (the paper has no counterpart).
 * higgs_launch_floor enqueues one kernel that does nothing, launched exactly like the product kernels (early start
 * permitted, `blocks` x `threads`, `shared_bytes` of dynamic shared memory <= 232448): a chain of them measures what a
 * chain of product launches costs before a byte moves.
 * higgs_selftest_wait runs the bounded wait of the small-batch kernel (which = 0) or of the tensor-core kernel
 * (which = 1) on a barrier that nothing arrives at, with no copy in flight, giving up after about `polls` polls
 * (<= 2^20): the kernel returns, result_out[0..1] (device int32[2]) is 0 for every wait that ran out, and
 * higgs_device_status() then reports HIGGS_ERR_TIMEOUT until cleared.  Nothing traps, faults or hangs.
 */
int higgs_launch_floor(int32_t blocks, int32_t threads, size_t shared_bytes, void* stream);
int higgs_selftest_wait(int32_t which, uint32_t polls, int32_t* result_out, void* stream);

/* Number of K ranges the product kernel assigns to different thread blocks for this shape and
 * batch (1 = not split), and whether those ranges meet in fp32 atomics.  For batches up to 16 two ranges are taken
 * by the two blocks of a thread-block cluster, which sum their partial results in a fixed order through
 * distributed shared memory; more than two accumulate with fp32 atomics into a cleared output (higgs_linear
 * clears it inside its rotation kernel, higgs_linear_prerotated with a memset), so the last bits of such a
 * result depend on timing: higgs_linear_uses_atomics returns 1 for exactly those calls.  The tensor-core path
 * (larger batches) sums the ranges of a tile in a fixed order inside a cluster too. */
int higgs_linear_uses_atomics(const higgs_desc* desc, int64_t B);
int higgs_linear_k_splits(const higgs_desc* desc, int64_t B);

/* Number of kernels one higgs_linear call enqueues for this shape and batch. */
int higgs_linear_launch_count(const higgs_desc* desc, int64_t B, int y_dtype);

/* ---- validation helpers (not on the hot path) --------------------------- */

/* Dequantisation to the original space (Appendix F, "Dequantization"):
 *   W_out[r][group i] = diag(sign) (H / sqrt(g)) ( scale[r][i] * G[codes of (r, i)] ),
 * the matrix the quantised layer stands for, so that y == x W_out^T up to rounding.
 *   packed, scales, grid : device, as written by higgs_quantize / passed to higgs_linear
 *   W_out                : device [N][K] row-major, w_dtype in {HIGGS_F32, HIGGS_BF16}
 *   workspace            : device, higgs_workspace_bytes(desc, HIGGS_OP_QUANTIZE, 0) bytes
 *                          (the canonical codes), 256-byte aligned
 * Errors as higgs_quantize.  Asynchronous on `stream`.                        */
int higgs_dequantize(const higgs_desc* desc, const void* packed, const void* scales, const float* grid,
                     void* W_out, int w_dtype, void* workspace, size_t workspace_bytes, void* stream);

/* ---- dynamic bit widths (Section 5) ------------------------------------------------------------------------ */

/* "Measuring Grid Parameters": one entry of the database of per-layer errors.  For the layer W quantised as
 * (packed, scales, grid) it accumulates, without materialising the dequantised matrix,
 *   sums_out[0] = || W^ - W ||_F^2,   sums_out[1] = || W ||_F^2,   sums_out[2] = t^2 = sums_out[0] / sums_out[1]
 * (device, three doubles, 8-byte aligned; t^2 = 0 for an all-zero layer): t^2 is the relative error of the linearity
 * theorem (Appendix E shows it equals the grid's expected squared error for Gaussian-like rotated weights).
 * W: device [N][K], w_dtype in {HIGGS_F32, HIGGS_BF16}; workspace as for higgs_dequantize.  Asynchronous.    */
int higgs_layer_error(const higgs_desc* desc, const void* W, int w_dtype, const void* packed, const void* scales,
                      const float* grid, double* sums_out, void* workspace, size_t workspace_bytes, void* stream);

/* Algorithm 1 for ANY grid (1 <= p <= 4, 1 <= n <= 4096, n need not be a power of two): the encoder for the grids
 * the paper evaluates beside the kernel-supported ones, e.g. (p, n) = (3, 830), (2, 88), (2, 361), (1, 19)
 * ("Experiment Configurations"), and the error-database entry of such a grid in the same pass.  No product
 * kernel reads this output.
 *   W          : device [N][K] row-major, w_dtype in {HIGGS_F32, HIGGS_BF16}; K a multiple of 1024 (the group size)
 *   grid       : device [n][p] fp32
 *   codes_out  : device [N][K/1024][T] uint16, T = higgs_general_tuples(p) = ceil(1024 / p); code t of a group covers
 *                rotated coordinates [t p, (t+1) p).  When p does not divide 1024 the last tuple is completed with
 *                zeros and matched on all p coordinates; its completed coordinates are dropped on reconstruction.
 *   scales_out : device [N][K/1024] fp16, ROW-major (not the product kernels' tile-major order): ||w|| / sqrt(1024)
 *   sums_out   : device, three doubles, optional: || W^ - W ||_F^2 (with the fp16 scale), || W ||_F^2 and their
 *                ratio t^2; cleared by the call.
 * HIGGS_ERR_UNSUPPORTED for p, n or K outside the above; HIGGS_ERR_INVALID_ARG for null pointers.  Asynchronous.  */
int higgs_general_tuples(int p);
int higgs_quantize_general(int p, int n, int64_t N, int64_t K, uint64_t rht_seed, const void* W, int w_dtype,
                           const float* grid, uint16_t* codes_out, void* scales_out, double* sums_out, void* stream);

/* Eq. 4: choose option j_l in [0, num_options) for every layer l, minimising  sum_l alpha[l] * t2[l][j_l]  subject
 * to  sum_l bits(j_l) * sizes[l] <= budget * sum_l sizes[l].  Exact (dynamic programming over the integer budget;
 * ties: lowest option index, then lowest total size).  HOST function, host pointers, no GPU involved.
 *   alpha[num_layers], t2[num_layers][num_options]  (row-major)
 *   bits64[num_options] : bits per weight of every option in units of 1/64 bit (a 16-bit scale per 1024 weights
 *                         is exactly 1/64 bit, so "4.02 bits" is 257); budget64: the target in the same unit
 *   sizes[num_layers]   : number of weights of every layer
 *   choice_out[num_layers], objective_out (optional)
 * HIGGS_ERR_UNSUPPORTED if no assignment fits the budget, HIGGS_ERR_WORKSPACE if the table
 * (num_layers x budget in reduced units) would exceed 2e9 entries.                                             */
int higgs_allocate_bits(int32_t num_layers, int32_t num_options, const double* alpha, const double* t2,
                        const int32_t* bits64, const int64_t* sizes, int64_t budget64, int32_t* choice_out,
                        double* objective_out);

/* The transform alone on `rows` rows of length K: out[r] = RHT of x[r] per
 * group (Algorithm 1 / Appendix F).  x_dtype in {HIGGS_F32, HIGGS_BF16};
 * out is device [rows][K] fp32; normalised != 0 divides by sqrt(g).        */
int higgs_rht(const higgs_desc* desc, const void* x, int x_dtype, int64_t rows,
              float* out, int normalised, void* stream);

/* Canonical codes ([N][K/p] bytes, device, 16-byte aligned) -> packed stream, and back.  They
 * let codes produced elsewhere (e.g. by a reference encoder) be fed to
 * higgs_linear, and the packed output of higgs_quantize be inspected.       */
int higgs_pack_codes(const higgs_desc* desc, const uint8_t* canonical, void* packed_out, void* stream);
int higgs_unpack_codes(const higgs_desc* desc, const void* packed, uint8_t* canonical_out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* HIGGS_H_ */
