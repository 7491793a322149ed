// Large-batch product in the rotated space (Appendix F, "Rotating Activations") on the 5th-generation tensor
// cores:  y[b][r] = sum_i scale[r][i] * sum_t < G[code[r][i][t]], x+[b][i][2t:2t+2] >  for 17 <= B tokens.
// Here the path is a dense contraction, so it runs as tcgen05.mma with the accumulator in tensor memory (TMEM).
//
// One block computes a 128-row x BN-token tile of y over a slice of K ("swap-AB": the weights are the M = 128 side).
//   producer warps   stream, per 64 inputs, the codes of the 128 rows (8 bulk copies of 512 B, a deep ring: they
//                    are the HBM stream) and, per 64/128/256 inputs, the tile of rotated activations (one bulk copy,
//                    from L2) into shared memory (TMA, cp.async.bulk + mbarrier);
//   16 dequant warps each thread owns one row of the tile: it turns the row's 32 code bytes of a 64-input step into
//                    table lookups (fp16 pairs), multiplies by the row's group scale and writes them with tcgen05.st
//                    straight into the TMEM columns the MMA reads as its A operand - dequantisation is fused into
//                    the operand load and the dequantised weights never touch shared or global memory.  The four
//                    warp groups fill the four quarters of one 256-input A stage at the same time;
//   MMA warp         one elected lane issues sixteen tcgen05.mma (M=128, N=BN, K=16, A from TMEM, B through a
//                    shared-memory descriptor) per A stage - one barrier wait per 256 inputs keeps the issuing
//                    warp's serial bookkeeping off the critical path - and commits them to the mbarriers that free
//                    the stages;
//   epilogue         all dequant warps read the fp32 accumulator with tcgen05.ld and park it in shared memory, from
//                    where y is written in 512-byte runs (or the cluster sums the K slices).
// Layers with few row tiles split K over the blocks of a thread-block cluster (grid z): every block parks its
// partial tile in its own shared memory, and after a cluster barrier block z sums the partials of "its" token
// columns through distributed shared memory in a fixed order and writes them - no atomics, no zeroing, and the
// result does not depend on timing.
// The group scale is folded into the fp16 A operand (relative rounding 2^-11, the same size as the rounding of the
// table entry itself), so one accumulation runs over all of K.  Every mbarrier wait is bounded; TMEM is always
// released.
#include "common.cuh"

#include <cuda.h>

namespace higgs {

__device__ int g_tc_status = 0;


namespace {

struct TcParams {
    const uint8_t* packed;   // packed code stream (byte format)
    const __half* scales;    // tile-major scales [N/16][K/g][16]
    const float* grid;       // [n][p]
    const __half* xdag;      // rotated activations, blocked: [batch tile][K/64][BN/8][8 k-cores][8 tokens][8 inputs]
    void* y;                 // [B][ldy]
    void* y_more[kMaxGather - 1];   // the same window on other devices (gathered output), n_more of them
    int n_more;
    int64_t N, K, ldy;
    int B, BN, n, p, y_mode; // y_mode 0: fp32, 1: bf16
    int bits;                // log2(n)
    int ksplit;              // K slices (= cluster size along z); each a multiple of 256 inputs
};

constexpr uint32_t kTcSmem = 232448;
constexpr int kTcGroups = 4;                 // dequant warp groups (4 warps each, one per TMEM lane quadrant)
constexpr int kTcBStages = 3;                // activation-tile stages in shared memory (at most 32 KB each)
constexpr int kTcMaxCodeStages = 32;         // code stages in shared memory (4 KB each), below and above the table
constexpr int kTcDequantWarps = 4 * kTcGroups;
constexpr int kTcThreads = (3 + kTcDequantWarps) * 32;
// a code stage: byte formats 128 rows x 64 inputs (4 KB, one step); six-bit format 128 rows x 128 inputs (6 KB, two steps:
// its three bit planes cover two neighbouring 64-input blocks)
constexpr uint32_t kTcWait = 1u << 22;
// TMEM columns: [0, BN) accumulator; A stages of 128 columns (256 inputs) from column 128 (BN <= 128: three stages)
// or 256 (two stages).
constexpr uint32_t kTcAStageCols = 128;
constexpr int kTcMaxSplit = 8;               // K slices = blocks per cluster (8 is the portable limit)

__device__ __forceinline__ uint32_t t_lds32(uint32_t a) { uint32_t v; asm("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(a)); return v; }
__device__ __forceinline__ uint4 t_lds128(uint32_t a) {
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
    return v;
}
__device__ __forceinline__ void t_mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void t_mbar_arrive(uint32_t bar) {
    asm volatile("{ .reg .b64 st; mbarrier.arrive.shared::cta.b64 st, [%0]; }" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void t_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("{ .reg .b64 st; mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1; }" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait, 1 when the phase completed, 0 when `limit` polls ran out.  The loop lives inside one asm statement and
// callers never branch on the result inside their main loops (they OR the failures into a flag and shrink the limit
// of later waits to one poll): a data-dependent exit from the loop that issues tcgen05.mma or bulk copies makes
// every such instruction several times more expensive to issue (measured: 16 -> 50 cycles per MMA).
__device__ __forceinline__ uint32_t t_wait(uint32_t bar, uint32_t parity, uint32_t limit) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\t.reg .u32 n;\n\tmov.u32 n, 0;\n\t"
                 "T_WAIT_LOOP:\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "@p bra T_WAIT_DONE;\n\t"
                 "add.u32 n, n, 1;\n\t"
                 "setp.lt.u32 p, n, %3;\n\t"
                 "@p bra T_WAIT_LOOP;\n\t"
                 "setp.ne.u32 p, n, n;\n\t"
                 "T_WAIT_DONE:\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity), "r"(limit) : "memory");
    return ok;
}
__device__ __forceinline__ uint32_t t_limit(uint32_t bad) { return bad ? 1u : kTcWait; }
// A role whose wait ran out reports it: the block's abort flag (read by the K-split reduction) and the status word.
__device__ __forceinline__ void t_report(uint32_t bad, volatile int* abort_flag) {
    if (bad) {
        *abort_flag = 1;
        atomicExch(&g_tc_status, (int)HIGGS_ERR_TIMEOUT);
    }
}
__device__ __forceinline__ void t_bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// One tiled TMA copy: the box (64 x 8-byte elements = one 512-byte block, 8 row tiles) at element column x, row tile y
// of the packed stream viewed as a 2-D tensor [N/16 row tiles][K x 8 bytes]; lands as [8][512 B] in shared memory.
__device__ __forceinline__ void t_tensor_load(uint32_t dst, const CUtensorMap* map, int32_t x, int32_t y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major operand without swizzle: 8-row x 16-byte core matrices, the two
// K-adjacent cores of an MMA step `lbo` bytes apart, cores adjacent along N `sbo` bytes apart.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    const uint64_t lo = (uint64_t)((addr & 0x3ffffu) >> 4) | ((uint64_t)(lbo >> 4) << 16);
    const uint64_t hi = (uint64_t)(sbo >> 4) | (1ull << 14);     // bits 46-47: descriptor version 1; layout type 0
    return lo | (hi << 32);
}
// D[tmem] (+)= A[tmem] * B[smem descriptor], one thread issues
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n\t}\n"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u) : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
          "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
          "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,"
        "%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}

// FB = 64-input steps per activation-tile stage (4, 2, 1 for BN <= 64, <= 128, <= 256: a stage is at most 32 KB).  It is a
// template parameter so that the MMA warp's loop body is straight-line code.
// FMT: 0 = byte format, 1 = six-bit planes, 2 = nibble pairs (p=2 n=16, p=1 n=4), 3 = 8-bit scalar codes (p=1 n=256).
template <int FB, int FMT>
__global__ void __launch_bounds__(kTcThreads, 1) linear_tc_kernel(const TcParams prm, const __grid_constant__ CUtensorMap code_map) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // ---- shared memory map ----
    //   [base, base+2 KB)    mbarriers, TMEM base address, abort flag
    //   [base+2 KB, lut)     code stages, region A (4 KB each): deep, because the codes are the HBM stream
    //   [lut, lut+64 KB)     lookup table, 256-byte rows (bytes 0..127 = the entry replicated per lane)
    //   [lut+64 KB, ...)     three activation-tile stages (FB x BN x 128 bytes each; they come from L2)
    //   [..., end)           code stages, region B (whatever the activation stages leave: 52 KB for BN <= 128)
    //   after the main loop: [base+2 KB, +BN x 512 B) the block's (partial) output tile, [token][row] fp32
    // Three rings: codes (freed when the four dequant warps of a step have read them), activation tiles and the
    // A operand in TMEM (both freed by tcgen05.commit when the MMAs that read them are done).
    const uint32_t base = (uint32_t)__cvta_generic_to_shared(smem_raw);
    const uint32_t lut = (base + 2048u + 0xffffu) & ~0xffffu;
    const uint32_t bars = base;
    auto code_full = [&](int s) { return bars + 8u * (uint32_t)s; };
    auto code_empty = [&](int s) { return bars + 8u * (uint32_t)(32 + s); };
    auto b_full = [&](int s) { return bars + 8u * (uint32_t)(64 + s); };
    auto b_free = [&](int s) { return bars + 8u * (uint32_t)(68 + s); };
    auto a_full = [&](int s) { return bars + 8u * (uint32_t)(72 + s); };
    auto a_free = [&](int s) { return bars + 8u * (uint32_t)(76 + s); };
    const uint32_t d_full = bars + 8u * 80u;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_raw + 1024);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_raw + 1032);
    constexpr bool SIX = FMT == 1, NIB = FMT == 2, B8 = FMT == 3;
    // bytes of the block's 128 rows in one code stage: 512 B per row tile and 64 inputs (byte format), 768 B per 128
    // inputs (six-bit), 256 B (nibble), 1 KB (8-bit)
    constexpr uint32_t kTcCodeStage = SIX ? 6144u : NIB ? 2048u : B8 ? 8192u : 4096u;
    constexpr int SPS = SIX ? 2 : 1;                         // 64-input steps per code stage
    const uint32_t code0 = base + 2048u;
    const uint32_t b_stage_bytes = (uint32_t)FB * (uint32_t)prm.BN * 128u;
    const uint32_t code1 = lut + 65536u + (uint32_t)kTcBStages * b_stage_bytes;      // region B
    int nA = (int)((lut - code0) / kTcCodeStage);
    if (nA > 16) nA = 16;
    int nB = (int)((base + kTcSmem - code1) / kTcCodeStage);
    if (nB > kTcMaxCodeStages - nA) nB = kTcMaxCodeStages - nA;
    const int CS = nA + nB;
    auto code_stage = [&](int s) { return s < nA ? code0 + (uint32_t)s * kTcCodeStage : code1 + (uint32_t)(s - nA) * kTcCodeStage; };
    auto b_stage = [&](int s) { return lut + 65536u + (uint32_t)s * b_stage_bytes; };

    const int BN = prm.BN;
    const int ksplit = prm.ksplit;
    const int kz = blockIdx.z;                               // K slice = rank in the cluster (cluster dims 1 x 1 x ksplit)
    const int ksteps_all = (int)(prm.K / 64);
    const int ksteps = ksteps_all / ksplit;                  // 64-input steps of this block, a multiple of 4
    const int kstep0 = kz * ksteps;
    const int nsuper = ksteps >> 2;                          // A stages (256 inputs) of this block
    const int64_t row0 = (int64_t)blockIdx.x * 128;
    const int bt = blockIdx.y;
    const uint32_t b_step_bytes = (uint32_t)BN * 128u;
    const int tile0 = (int)(row0 / 16);                      // first 16-row tile of this block
    const int AS = BN <= 128 ? 3 : 2;                        // A stages in TMEM
    const uint32_t acol0 = BN <= 128 ? 128u : 256u;

    // ---- prologue ----
    // (1) the table's source: the grid loads are in flight while everything else is set up.  Warp w fills rows
    //     4 (w + 19 r) .. + 3; a row's 128 bytes are written by eight lanes with one 16-byte store each.
    constexpr int kW = kTcThreads / 32;
    constexpr int kQuads = (64 + kW - 1) / kW;
    float ent_lo[kQuads], ent_hi[kQuads];
#pragma unroll
    for (int r = 0; r < kQuads; ++r) {
        const int idx = 4 * (warp + r * kW) + (lane >> 3);
        ent_lo[r] = 0.f; ent_hi[r] = 0.f;
        if (idx < 256) {
            if (B8) {
                ent_lo[r] = ent_hi[r] = __ldg(prm.grid + idx);              // one input per index: the value in both halves
            } else if (prm.p == 2) {
                const float2 gp = __ldg(reinterpret_cast<const float2*>(prm.grid) + (idx & (prm.n - 1)));
                ent_lo[r] = gp.x; ent_hi[r] = gp.y;
            } else {
                ent_lo[r] = __ldg(prm.grid + (idx & (prm.n - 1)));          // two p=1 codes per table index
                ent_hi[r] = __ldg(prm.grid + ((idx >> prm.bits) & (prm.n - 1)));
            }
        }
    }
    // The code ring needs one stage per warp group; the block's shared-memory window always leaves room for more, but
    // a window that did not would be reported, not run.
    int role = warp;
    if (CS < kTcGroups) role = -1;
    // (2) barriers, each ring by the warp that produces into it; the code producer starts the weight stream (which
    //     depends on nothing) before the block-wide barrier: the first CS stages need no wait.
    int code_issued = 0;
    uint32_t elected;
    asm volatile("{ .reg .pred p; elect.sync _|p, 0xffffffff; selp.u32 %0, 1, 0, p; }" : "=r"(elected));
    if (warp == 0) {
        t_mbar_init(code_full(lane), 1);
        t_mbar_init(code_empty(lane), 4 * SPS);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (role == 0) {
            const int nstage = ksteps / SPS;
            const int n0 = nstage < CS ? nstage : CS;
            for (int j = 0; j < n0; ++j) {
                if (elected) {
                    t_mbar_expect_tx(code_full(j), kTcCodeStage);
                    t_tensor_load(code_stage(j), &code_map, (kstep0 / SPS + j) * (int)(kTcCodeStage / 64u), tile0, code_full(j));
                }
                __syncwarp();
            }
            code_issued = n0;
        }
    } else if (warp == 1) {
        if (lane < 4) { t_mbar_init(a_full(lane), kTcDequantWarps); t_mbar_init(a_free(lane), 1); }
        if (lane == 4) t_mbar_init(d_full, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        // one warp allocates all 512 TMEM columns (one block per SM, so nobody else wants them)
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(base + 1024u), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    } else if (warp == 2) {
        if (lane < 4) { t_mbar_init(b_full(lane), 1); t_mbar_init(b_free(lane), 1); }
        if (lane == 4) {
            *abort_flag = 0;
            if (role < 0) { *abort_flag = 1; atomicExch(&g_tc_status, (int)HIGGS_ERR_TIMEOUT); }
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    pdl_trigger();
    // (3) the table
#pragma unroll
    for (int r = 0; r < kQuads; ++r) {
        const int idx = 4 * (warp + r * kW) + (lane >> 3);
        __half2 h = __floats2half2_rn(ent_lo[r], ent_hi[r]);
        const uint32_t e = *reinterpret_cast<uint32_t*>(&h);
        if (idx < 256) *reinterpret_cast<uint4*>(smem_raw + (lut - base) + idx * 256 + (lane & 7) * 16) = make_uint4(e, e, e, e);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (role == 0) {
        // =============================== code producer (weights: no dependency on earlier kernels) ===============
        // (whole warp in the loop, one elected lane issues: bulk copies take warp-uniform operands; the first stages
        // were issued in the prologue)
        int issued = code_issued;
        int s = issued == CS ? 0 : issued, it = issued == CS ? 1 : 0;
        uint32_t bad = 0;
        for (int j = issued; j < ksteps / SPS; ++j) {
            bad |= t_wait(code_empty(s), (uint32_t)((it & 1) ^ 1), t_limit(bad)) ^ 1u;
            if (elected) {
                t_mbar_expect_tx(code_full(s), kTcCodeStage);
                t_tensor_load(code_stage(s), &code_map, (kstep0 / SPS + j) * (int)(kTcCodeStage / 64u), tile0, code_full(s));
            }
            ++issued;
            const bool wrap = s + 1 == CS;
            s = wrap ? 0 : s + 1;
            it += wrap ? 1 : 0;
            __syncwarp();
        }
        // never leave with copies in flight: wait (bounded) for the last stages issued
        for (int j = issued > CS ? issued - CS : 0; j < issued; ++j)
            bad |= t_wait(code_full(j % CS), (uint32_t)((j / CS) & 1), t_limit(bad)) ^ 1u;
        t_report(bad, abort_flag);
    } else if (role == 2) {
        // =============================== activation-tile producer ===============================
        pdl_wait();            // the rotated activations are the previous kernel's output
        int issued = 0;
        const int nb = ksteps / FB;
        const uint32_t bytes = b_step_bytes * (uint32_t)FB;
        const __half* xsrc = prm.xdag + ((int64_t)bt * ksteps_all + kstep0) * BN * 64;
        int s = 0, it = 0;
        uint32_t bad = 0;
        for (int t = 0; t < nb; ++t) {
            bad |= t_wait(b_free(s), (uint32_t)((it & 1) ^ 1), t_limit(bad)) ^ 1u;
            if (elected) {
                t_mbar_expect_tx(b_full(s), bytes);
                t_bulk_load(b_stage(s), xsrc + (int64_t)t * FB * BN * 64, bytes, b_full(s));
            }
            ++issued;
            const bool wrap = s + 1 == kTcBStages;
            s = wrap ? 0 : s + 1;
            it += wrap ? 1 : 0;
            __syncwarp();
        }
        for (int t = issued > kTcBStages ? issued - kTcBStages : 0; t < issued; ++t)
            bad |= t_wait(b_full(t % kTcBStages), (uint32_t)((t / kTcBStages) & 1), t_limit(bad)) ^ 1u;
        t_report(bad, abort_flag);
    } else if (role == 1) {
        // =============================== MMA issuer ===============================
        // The whole warp runs the loop so that addresses and descriptors stay warp-uniform (tcgen05.mma takes its
        // operands from uniform registers); one elected lane issues.  Per A stage (256 inputs): one wait for the
        // sixteen dequant warps, one wait per activation-tile stage, sixteen MMAs.
        const uint32_t idesc = (1u << 4) | ((uint32_t)(BN >> 3) << 17) | (8u << 24);   // f32 accumulate, f16 x f16, K-major, M=128
        int sa = 0, ua = 0;            // A stage and its use count
        int sb = 0, ub = 0;            // activation-tile stage and its use count
        uint32_t bad = 0;
        const uint64_t b_desc0 = smem_desc(b_stage(0), 128u, 1024u);
        for (int S = 0; S < nsuper; ++S) {
            bad |= t_wait(a_full(sa), (uint32_t)(ua & 1), t_limit(bad)) ^ 1u;
            tc_fence_after();
            const uint32_t a_stage = tmem + acol0 + kTcAStageCols * (uint32_t)sa;
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                if (h % FB == 0) {
                    bad |= t_wait(b_full(sb), (uint32_t)(ub & 1), t_limit(bad)) ^ 1u;
                    tc_fence_after();
                }
                // addresses and descriptors are computed by the whole warp; only the instruction is issued by one lane
                const uint32_t a_addr = a_stage + 32u * (uint32_t)h;
                const uint64_t b_desc = b_desc0 + (uint64_t)(((uint32_t)sb * b_stage_bytes + (uint32_t)(h % FB) * b_step_bytes) >> 4);
                const uint32_t acc = (uint32_t)((S | h) != 0);
                if (elected) {
                    tc_mma(tmem, a_addr, b_desc, idesc, acc);
                    tc_mma(tmem, a_addr + 8u, b_desc + 16u, idesc, 1u);      // + 256 bytes in the address field
                    tc_mma(tmem, a_addr + 16u, b_desc + 32u, idesc, 1u);
                    tc_mma(tmem, a_addr + 24u, b_desc + 48u, idesc, 1u);
                    if (h % FB == FB - 1) tc_commit(b_free(sb));      // arrives when the MMAs issued so far are done
                }
                if (h % FB == FB - 1) {
                    const bool wrap = sb + 1 == kTcBStages;
                    sb = wrap ? 0 : sb + 1;
                    ub += wrap ? 1 : 0;
                }
            }
            if (elected) tc_commit(a_free(sa));
            const bool wrap = sa + 1 == AS;
            sa = wrap ? 0 : sa + 1;
            ua += wrap ? 1 : 0;
            __syncwarp();
        }
        if (elected) tc_commit(d_full);       // -> the accumulator is final
        t_report(bad, abort_flag);
    } else if (role >= 3) {
        // =============================== dequant warps (then epilogue) ===============================
        // A warp may touch only the TMEM lanes 32 (warp % 4) .. +31; the four warps sharing a quadrant (warp groups
        // sg = 0..3) take the four 64-input quarters of each A stage.
        const int q = warp & 3, sg = (warp - 3) >> 2;
        const int i = 32 * q + lane;               // row of the tile = TMEM lane
        const int rtl = i >> 4, g = i & 7, h = (i >> 3) & 1;
        const uint32_t lut_lane = lut + lane * 4;
        const uint32_t sel0 = 0x7604u + ((uint32_t)h << 4), sel1 = 0x7624u + ((uint32_t)h << 4);   // bytes h and h+2 of a word
        const int rot = g >> 1;                    // chunk rotation that makes the 16-byte code loads conflict-free
        const int groups = (int)(prm.K / kGroup);
        const __half* sc_row = prm.scales + ((row0 / 16 + rtl) * groups) * 16 + (i & 15);
        const uint32_t t_lane = tmem + ((uint32_t)(32 * q) << 16);
        // byte formats: this row's words are the 16-byte chunks of lanes (g, t) of its row tile; six-bit: word 2 (4g + t) +
        // (step & 1) of each of the tile's three 256-byte planes
        // nibble format: the 8-byte chunks of lanes (g, t = 0..3) are 32 contiguous bytes; 8-bit format: the 16-byte chunks
        // of lanes (g, t) in each 512-byte half of the row tile's 1 KB block
        const uint32_t code_off = SIX ? (uint32_t)(rtl * 768 + g * 32 + (sg & 1) * 4) : NIB ? (uint32_t)(rtl * 256 + g * 32)
                                : B8 ? (uint32_t)(rtl * 1024 + g * 64) : (uint32_t)(rtl * 512 + g * 64);
        const int tx = rtl & 1;                    // six-bit: odd row tiles visit the lanes t in the order t ^ 1 (bank conflicts)
        int cur_group = -1;
        uint32_t sc2 = 0;
        uint32_t bad = 0;
        int sa = 0, ua = 0;
        int cs = (sg / SPS) % CS, ucs = 0;         // code stage of step 4 S + sg and its use count (CS >= 4)
        for (int S = 0; S < nsuper; ++S) {
            const int jg = kstep0 + 4 * S + sg;    // 64-input step of the layer
            bad |= t_wait(code_full(cs), (uint32_t)(ucs & 1), t_limit(bad)) ^ 1u;
            if ((jg >> 4) != cur_group) {          // new group of 1024 inputs: this row's scale
                cur_group = jg >> 4;
                const __half sc = sc_row[cur_group * 16];
                const __half2 s2 = __half2half2(sc);
                sc2 = *reinterpret_cast<const uint32_t*>(&s2);
            }
            uint4 c4[4] = {};                      // c4[t] = the four index words (steps m = 0..3) of lane (g, t)
            uint32_t a[32];
            auto unrotate = [&]() {                // chunk t was loaded by instruction (t - rot) & 3
                if (rot & 1) { const uint4 t0 = c4[0]; c4[0] = c4[3]; c4[3] = c4[2]; c4[2] = c4[1]; c4[1] = t0; }
                if (rot & 2) { uint4 t0 = c4[0]; c4[0] = c4[2]; c4[2] = t0; t0 = c4[1]; c4[1] = c4[3]; c4[3] = t0; }
            };
            if (B8) {
                // 8-bit scalar codes: a register (two consecutive inputs of the row) is halfword h of word 2m + kh of lane
                // (g, t) - two code bytes, two lookups (a table entry carries its value in both halves).  Words 0..3 of
                // every lane sit in the first 512-byte half of the row tile's block (steps m = 0, 1), words 4..7 in the second.
                const uint32_t selA = 0x7604u + ((uint32_t)(2 * h) << 4), selB = 0x7604u + ((uint32_t)(2 * h + 1) << 4);
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
#pragma unroll
                    for (int jj = 0; jj < 4; ++jj)
                        c4[jj] = t_lds128(code_stage(cs) + code_off + (uint32_t)(hh * 512) + (uint32_t)(((jj + rot) & 3) * 16));
                    unrotate();
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
#pragma unroll
                        for (int r = 0; r < 4; ++r) {          // r = 2 (m & 1) + kh
                            const uint32_t w = r == 0 ? c4[t].x : r == 1 ? c4[t].y : r == 2 ? c4[t].z : c4[t].w;
                            const uint32_t l0 = t_lds32(__byte_perm(w, lut_lane, selA));
                            const uint32_t l1 = t_lds32(__byte_perm(w, lut_lane, selB));
                            const uint32_t e = __byte_perm(l0, l1, 0x7610);
                            const __half2 pr = __hmul2(*reinterpret_cast<const __half2*>(&e), *reinterpret_cast<const __half2*>(&sc2));
                            a[(2 * hh + (r >> 1)) * 8 + (r & 1) * 4 + t] = *reinterpret_cast<const uint32_t*>(&pr);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) t_mbar_arrive(code_empty(cs));     // every code word has been looked up: hand the stage back
                cs += 4 / SPS;
                if (cs >= CS) { cs -= CS; ++ucs; }
            } else {
            if (NIB) {
                // nibble pairs: byte 2m + kh of lane (g, t) holds the codes of row halves 0 (low nibble) and 1 (high nibble);
                // the row's eight nibbles per lane become the bytes of two index words.  The two 16-byte loads are issued in
                // the order that keeps the eight g of a warp on different banks.
                const bool swp = (g & 4) != 0;
                const uint4 f0 = t_lds128(code_stage(cs) + code_off + (swp ? 16u : 0u));
                const uint4 f1 = t_lds128(code_stage(cs) + code_off + (swp ? 0u : 16u));
                const uint4 lo = swp ? f1 : f0, hi = swp ? f0 : f1;        // lanes t = 0, 1 and t = 2, 3
                const uint32_t sh = (uint32_t)(4 * h);
                c4[0] = make_uint4((lo.x >> sh) & 0x0f0f0f0fu, (lo.y >> sh) & 0x0f0f0f0fu, 0u, 0u);
                c4[1] = make_uint4((lo.z >> sh) & 0x0f0f0f0fu, (lo.w >> sh) & 0x0f0f0f0fu, 0u, 0u);
                c4[2] = make_uint4((hi.x >> sh) & 0x0f0f0f0fu, (hi.y >> sh) & 0x0f0f0f0fu, 0u, 0u);
                c4[3] = make_uint4((hi.z >> sh) & 0x0f0f0f0fu, (hi.w >> sh) & 0x0f0f0f0fu, 0u, 0u);
            } else if (!SIX) {
                // the 16-byte chunks of lanes (g, t = 0..3) of row tile rtl; instruction jj reads chunk (jj + rot) & 3
                // so that the eight g of a warp hit eight different bank groups
#pragma unroll
                for (int jj = 0; jj < 4; ++jj)
                    c4[jj] = t_lds128(code_stage(cs) + code_off + (uint32_t)(((jj + rot) & 3) * 16));
            } else {
                uint32_t w0[4], w1[4], w2[4];
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const uint32_t addr = code_stage(cs) + code_off + (uint32_t)((t ^ tx) * 8);
                    w0[t] = t_lds32(addr);
                    w1[t] = t_lds32(addr + 256u);
                    w2[t] = t_lds32(addr + 512u);
                }
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    // low nibbles: slot 4m + a at bit 8a + 4(m & 1) of word m >> 1; high bit pairs: bit 8a + 2m of word 2.
                    // (x & 0x0f0f0f0f) | (y & 0xf0f0f0f0): bits 6-7 of every byte are don't-care (the table repeats)
                    uint32_t r0, r1, r2, r3;
                    asm("lop3.b32 %0, %1, %2, 0x0f0f0f0f, 0xe4;" : "=r"(r0) : "r"(w0[t]), "r"(w2[t] << 4));
                    asm("lop3.b32 %0, %1, %2, 0x0f0f0f0f, 0xe4;" : "=r"(r1) : "r"(w0[t] >> 4), "r"(w2[t] << 2));
                    asm("lop3.b32 %0, %1, %2, 0x0f0f0f0f, 0xe4;" : "=r"(r2) : "r"(w1[t]), "r"(w2[t]));
                    asm("lop3.b32 %0, %1, %2, 0x0f0f0f0f, 0xe4;" : "=r"(r3) : "r"(w1[t] >> 4), "r"(w2[t] >> 2));
                    c4[t] = make_uint4(r0, r1, r2, r3);
                }
                if (tx) { uint4 t0 = c4[0]; c4[0] = c4[1]; c4[1] = t0; t0 = c4[2]; c4[2] = c4[3]; c4[3] = t0; }
            }
            __syncwarp();
            if (lane == 0) t_mbar_arrive(code_empty(cs));     // the code words are in registers: hand the stage back
            cs += 4 / SPS;
            if (cs >= CS) { cs -= CS; ++ucs; }
            if (!SIX && !NIB) unrotate();
#pragma unroll
            for (int m = 0; m < 4; ++m) {
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    uint32_t e0, e1;
                    if (NIB) {
                        // bytes 2 (m & 1) and 2 (m & 1) + 1 of index word m >> 1: input pairs 8m + t and 8m + 4 + t
                        const uint32_t w = (m >> 1) ? c4[t].y : c4[t].x;
                        e0 = t_lds32(__byte_perm(w, lut_lane, (m & 1) ? 0x7624u : 0x7604u));
                        e1 = t_lds32(__byte_perm(w, lut_lane, (m & 1) ? 0x7634u : 0x7614u));
                    } else {
                        const uint32_t w = m == 0 ? c4[t].x : m == 1 ? c4[t].y : m == 2 ? c4[t].z : c4[t].w;
                        // input pairs 8m + t (byte h) and 8m + 4 + t (byte h + 2) of the 64-input block
                        e0 = t_lds32(__byte_perm(w, lut_lane, sel0));
                        e1 = t_lds32(__byte_perm(w, lut_lane, sel1));
                    }
                    const __half2 p0 = __hmul2(*reinterpret_cast<const __half2*>(&e0), *reinterpret_cast<const __half2*>(&sc2));
                    const __half2 p1 = __hmul2(*reinterpret_cast<const __half2*>(&e1), *reinterpret_cast<const __half2*>(&sc2));
                    a[m * 8 + t] = *reinterpret_cast<const uint32_t*>(&p0);
                    a[m * 8 + 4 + t] = *reinterpret_cast<const uint32_t*>(&p1);
                }
            }
            }
            // the A stage must have been consumed by the MMAs that used it last
            bad |= t_wait(a_free(sa), (uint32_t)((ua & 1) ^ 1), t_limit(bad)) ^ 1u;   // (first use: the phase before the first)
            tc_fence_after();
            tc_st32(t_lane + acol0 + kTcAStageCols * (uint32_t)sa + 32u * (uint32_t)sg, a);   // column 8m + jj = input pair 8m + jj
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            tc_fence_before();
            __syncwarp();
            if (lane == 0) t_mbar_arrive(a_full(sa));
            if (++sa == AS) { sa = 0; ++ua; }
        }
        bad |= t_wait(d_full, 0u, t_limit(bad)) ^ 1u;
        t_report(bad, abort_flag);
        if (!bad) {
            tc_fence_after();
            // Park the fp32 tile in shared memory as [token][row] (all rings are idle: every MMA has completed, so
            // every copy has landed and every lookup has been done).  Without a K split it is written out from there in
            // 512-byte runs (one token's 128 rows per store instruction of a warp): storing straight from the
            // accumulator registers - 128 bytes per instruction, 32 instructions per thread - took 1.5-1.8 us per 32
            // token columns.  With a K split the cluster sums the parked tiles.
            for (int c0 = 32 * sg; c0 < BN; c0 += 32 * kTcGroups) {
                uint32_t d[32];
                tc_ld32(t_lane + (uint32_t)c0, d);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int r = 0; r < 32; ++r)
                    if (c0 + r < BN)
                        asm volatile("st.shared.b32 [%0], %1;" ::"r"(code0 + (uint32_t)(((c0 + r) * 128 + i) * 4)), "r"(d[r]) : "memory");
            }
        }
    }

    // ---- every role ends here, aborted or not: TMEM must be handed back ----
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
    if (ksplit == 1) {
        // the parked tile -> y: warp w writes token columns w, w + 16, ...; a lane holds four consecutive rows
        if (tid < 512 && !*abort_flag) {
            pdl_wait();            // y may still be read by the kernel before this one
            for (int c = warp; c < BN; c += 16) {
                const int b = bt * BN + c;
                if (b >= prm.B) break;
                uint32_t v0, v1, v2, v3;
                asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(v0), "=r"(v1), "=r"(v2), "=r"(v3)
                             : "r"(code0 + (uint32_t)((c * 128 + lane * 4) * 4)) : "memory");
                const int64_t o = (int64_t)b * prm.ldy + row0 + lane * 4;
                if (prm.y_mode == 0) {
                    const uint4 v = make_uint4(v0, v1, v2, v3);
                    *reinterpret_cast<uint4*>(static_cast<float*>(prm.y) + o) = v;
                    for (int pd = 0; pd < prm.n_more; ++pd)       // gathered output: the other devices' copies
                        *reinterpret_cast<uint4*>(static_cast<float*>(prm.y_more[pd]) + o) = v;
                } else {
                    const __nv_bfloat162 lo = __floats2bfloat162_rn(__uint_as_float(v0), __uint_as_float(v1));
                    const __nv_bfloat162 hi = __floats2bfloat162_rn(__uint_as_float(v2), __uint_as_float(v3));
                    const uint2 v = make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
                    *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(prm.y) + o) = v;
                    for (int pd = 0; pd < prm.n_more; ++pd)
                        *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(prm.y_more[pd]) + o) = v;
                }
            }
        }
    } else {
        // Cluster reduction in a fixed order: block kz owns the token columns [kz, kz+1) * BN / ksplit and sums the
        // partial tiles of all blocks of the cluster for them through distributed shared memory.
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
        const int cols = BN / ksplit;
        if (tid < 512 && !*abort_flag) {
            pdl_wait();            // y may still be read by the kernel before this one
            // warp w sums token columns w, w + 16, ... of this block's share; a lane holds four consecutive rows, so a
            // warp reads 512 contiguous bytes of every slice's tile and writes 512 contiguous bytes of y
            for (int cc = warp; cc < cols; cc += 16) {
                const int c = kz * cols + cc;
                const uint32_t local = code0 + (uint32_t)((c * 128 + lane * 4) * 4);
                float4 part[8];
#pragma unroll
                for (int r = 0; r < 8; ++r) {
                    part[r] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (r < ksplit) {
                        uint32_t remote;
                        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(r));
                        asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];"
                                     : "=f"(part[r].x), "=f"(part[r].y), "=f"(part[r].z), "=f"(part[r].w) : "r"(remote) : "memory");
                    }
                }
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int r = 0; r < 8; ++r) {            // slice order: fixed, so the sum is reproducible
                    if (r < ksplit) { acc.x += part[r].x; acc.y += part[r].y; acc.z += part[r].z; acc.w += part[r].w; }
                }
                const int b = bt * BN + c;
                if (b < prm.B) {
                    const int64_t o = (int64_t)b * prm.ldy + row0 + lane * 4;
                    if (prm.y_mode == 0) {
                        *reinterpret_cast<float4*>(static_cast<float*>(prm.y) + o) = acc;
                        for (int pd = 0; pd < prm.n_more; ++pd)
                            *reinterpret_cast<float4*>(static_cast<float*>(prm.y_more[pd]) + o) = acc;
                    } else {
                        const __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
                        const uint2 v = make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
                        *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(prm.y) + o) = v;
                        for (int pd = 0; pd < prm.n_more; ++pd)
                            *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(prm.y_more[pd]) + o) = v;
                    }
                }
            }
        }
        // nobody leaves while its shared memory may still be read
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    }
}

}  // namespace

namespace {

// Rotation of the activations (Appendix F) for the tensor-core path: four warps per (token, group) - the transform sits
// on the latency path between dependent launches -, output written in the blocked order the MMA's shared-memory
// descriptor expects, so that one stage (BN tokens x 64 inputs) is one contiguous run:
//   [batch tile][K/64][BN/8 token blocks][8 input cores][8 tokens][8 inputs] fp16.
// Warp q of the block owns inputs 256 q .. + 255 of the group, 8 consecutive ones per lane (one core-matrix row):
// butterflies over those 8 in registers, over the 32 lanes by shuffles, over the 4 warps through shared memory.
__global__ void __launch_bounds__(128) rht_activations_tc_kernel(const __nv_bfloat16* __restrict__ x, __half* __restrict__ xdag,
                                                                 int64_t B, int64_t K, uint64_t xi, int BN) {
    __shared__ __align__(16) float ex[4][256];
    const int lane = threadIdx.x & 31, q = threadIdx.x >> 5;
    const int64_t groups = K / kGroup;
    pdl_trigger();
    pdl_wait();
    const int64_t b = blockIdx.x / groups, gi = blockIdx.x % groups;       // grid = B * groups blocks
    const int64_t k0 = gi * kGroup + q * 256 + lane * 8;
    float v[8];
    {
        const uint4 q4 = __ldg(reinterpret_cast<const uint4*>(x + b * K + k0));
        const uint32_t w4[4] = {q4.x, q4.y, q4.z, q4.w};
        const uint32_t bits = (uint32_t)(sign_word(xi, (uint64_t)k0 >> 6) >> ((uint64_t)k0 & 63ull)) & 0xffu;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            v[2 * e] = __uint_as_float((w4[e] << 16) ^ (((bits >> (2 * e)) & 1u) << 31));
            v[2 * e + 1] = __uint_as_float((w4[e] & 0xffff0000u) ^ (((bits >> (2 * e + 1)) & 1u) << 31));
        }
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
    uint32_t w4[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const __half2 hh = __floats2half2_rn(o[2 * e] * 0.03125f, o[2 * e + 1] * 0.03125f);
        w4[e] = *reinterpret_cast<const uint32_t*>(&hh);
    }
    const int64_t bt = b / BN, nloc = b % BN;
    const int64_t off = ((bt * (K / 64) + k0 / 64) * BN * 64) + (nloc / 8) * 512 + ((k0 % 64) / 8) * 64 + (nloc % 8) * 8;
    *reinterpret_cast<uint4*>(xdag + off) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
}

}  // namespace

// Token-tile width of the tensor-core path for batch B: a multiple of 16, at most 256, balanced over the tiles.
int tc_batch_tile(int64_t B) {
    const int64_t tiles = (B + 255) / 256;
    const int64_t per = (B + tiles - 1) / tiles;
    return (int)((per + 15) / 16 * 16);
}

// The tensor-core path takes layers whose row count is a multiple of 128: every batch above 16, and batches
// 9..16 of layers with at least 4096 rows, 4096 inputs and 16 M weights (there the small-batch kernel is limited by the legacy
// mma.sync rate, two per lookup group; measured at 16 tokens: 4096 x 4096 8.7 us here against 11.6 us there, 8192 x 2048
// 8.1 against 7.6 (stays there), and 2048 x 8192 - few row tiles, K split over a cluster - takes 12.9 us here against 9.3 us there.
bool tc_eligible(const higgs_desc& d, int64_t B) {
    const Format f = format_of(d.p, d.n);
    if (!(d.N % 128 == 0 && d.N > 0 && f != Format::kNone)) return false;
    return B > 16 || (B > 8 && d.N >= 4096 && d.K >= 4096 && d.N * d.K >= ((int64_t)1 << 24));
}

size_t tc_workspace_bytes(const higgs_desc& d, int64_t B) {
    const int BN = tc_batch_tile(B);
    const int64_t tiles = (B + BN - 1) / BN;
    return (size_t)tiles * BN * d.K * 2;
}

// D1 for the tensor-core path: rotated activations in the blocked operand layout (tc_workspace_bytes() bytes).
int launch_rht_tc(const higgs_desc& d, const void* x, int64_t B, __half* xdag_tc, cudaStream_t st) {
    const int BN = tc_batch_tile(B);
    const int64_t blocks = B * (d.K / kGroup);              // four warps per (token, group)
    if (blocks > 0x7fffffff) return HIGGS_ERR_UNSUPPORTED;
    return cuda_status(launch_pdl(rht_activations_tc_kernel, dim3((unsigned)blocks), dim3(128), 0, st,
                                  static_cast<const __nv_bfloat16*>(x), xdag_tc, B, d.K, d.rht_seed, BN));
}

// K slices of the tensor-core product: as many (a power of two, at most 8) as keep the grid within one wave of
// clusters, every slice a multiple of 256 inputs and at least 512.
int tc_k_split(const higgs_desc& d, int64_t B) {
    const int BN = tc_batch_tile(B);
    const int64_t tiles = (d.N / 128) * ((B + BN - 1) / BN);
    int ks = 1;
    while (ks < kTcMaxSplit && tiles * (ks * 2) <= 128 && d.K % (256 * ks * 2) == 0 && d.K / (ks * 2) >= 512) ks *= 2;
    return ks;
}

namespace {

// cuTensorMapEncodeTiled through the runtime's driver-entry-point query (the library does not link libcuda).
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
    static const EncodeTiledFn fn = [] {       // initialised once (thread-safe)
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            return reinterpret_cast<EncodeTiledFn>(p);
        return static_cast<EncodeTiledFn>(nullptr);
    }();
    return fn;
}

// The packed byte stream of a layer as a 2-D tensor of 8-byte elements: row = 16-row tile (K x 8 bytes: K/64 blocks
// of 512 bytes), box = one block column of eight consecutive row tiles (the 128 rows of a thread block).
bool make_code_map(const higgs_desc& d, const void* packed, CUtensorMap* map) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    // per row tile (16 rows) an input takes 8 bytes (byte format), 6 (six-bit), 4 (nibble) or 16 (8-bit); a stage is
    // one 64-input block of the eight row tiles - for the six-bit format one 768-byte super-block (three bit planes of
    // two neighbouring blocks)
    const Format f = format_of(d.p, d.n);
    const cuuint64_t bpi = f == Format::kSixBit ? 6 : f == Format::kNibble ? 4 : f == Format::kByte8 ? 16 : 8;
    const cuuint64_t dims[2] = {(cuuint64_t)d.K * bpi / 8, (cuuint64_t)(d.N / 16)};
    const cuuint64_t strides[1] = {(cuuint64_t)d.K * bpi};
    const cuuint32_t box[2] = {f == Format::kSixBit ? 96u : f == Format::kNibble ? 32u : f == Format::kByte8 ? 128u : 64u, 8};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_INT64, 2, const_cast<void*>(packed), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// D2-D5 on the tensor cores, from activations rotated by launch_rht_tc for the same B.
int launch_linear_tc(const higgs_desc& d, const __half* xdag_tc, int64_t B, const void* packed, const void* scales,
                     const float* grid, void* y, int y_mode, cudaStream_t st, int64_t ldy, const GatherTargets* more) {
    if (more && more->count > kMaxGather - 1) return HIGGS_ERR_INVALID_ARG;
    const int BN = tc_batch_tile(B);
    const int64_t tiles = (B + BN - 1) / BN;
    static int configured[64] = {0};
    const int conf = device_once(configured, [] {
        const void* kernels[12] = {
            (const void*)linear_tc_kernel<1, 0>, (const void*)linear_tc_kernel<2, 0>, (const void*)linear_tc_kernel<4, 0>,
            (const void*)linear_tc_kernel<1, 1>, (const void*)linear_tc_kernel<2, 1>, (const void*)linear_tc_kernel<4, 1>,
            (const void*)linear_tc_kernel<1, 2>, (const void*)linear_tc_kernel<2, 2>, (const void*)linear_tc_kernel<4, 2>,
            (const void*)linear_tc_kernel<1, 3>, (const void*)linear_tc_kernel<2, 3>, (const void*)linear_tc_kernel<4, 3>};
        for (const void* k : kernels)
            if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTcSmem) != cudaSuccess) return -1;
        return 1;
    });
    if (conf < 0) return HIGGS_ERR_CUDA;
    CUtensorMap code_map;
    if (!make_code_map(d, packed, &code_map)) return HIGGS_ERR_CUDA;
    TcParams prm;
    prm.packed = static_cast<const uint8_t*>(packed);
    prm.scales = static_cast<const __half*>(scales);
    prm.grid = grid;
    prm.xdag = xdag_tc;
    prm.y = y;
    prm.n_more = more ? more->count : 0;
    for (int i = 0; i < kMaxGather - 1; ++i) prm.y_more[i] = (more && i < more->count) ? more->y[i] : nullptr;
    prm.N = d.N; prm.K = d.K; prm.ldy = ldy > 0 ? ldy : d.N;
    prm.B = (int)B; prm.BN = BN; prm.n = d.n; prm.p = d.p; prm.y_mode = y_mode;
    prm.bits = code_bits(d.n);
    prm.ksplit = tc_k_split(d, B);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(d.N / 128), (unsigned)tiles, (unsigned)prm.ksplit);
    cfg.blockDim = dim3(kTcThreads);
    cfg.dynamicSmemBytes = kTcSmem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.numAttrs = 1;
    if (prm.ksplit > 1) {      // the K slices of a tile form one thread-block cluster
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = 1;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = (unsigned)prm.ksplit;
        cfg.numAttrs = 2;
    }
    cfg.attrs = attr;
    // activation-tile stage = FB steps of BN x 128 bytes, at most 16 KB for BN <= 128 (so that the code ring gets the
    // rest of shared memory) and 32 KB for wider tiles
    const Format fmt = format_of(d.p, d.n);
    const int fi = fmt == Format::kSixBit ? 1 : fmt == Format::kNibble ? 2 : fmt == Format::kByte8 ? 3 : 0;
    typedef void (*TcKernel)(const TcParams, const CUtensorMap);
    static const TcKernel table[3][4] = {
        {linear_tc_kernel<4, 0>, linear_tc_kernel<4, 1>, linear_tc_kernel<4, 2>, linear_tc_kernel<4, 3>},
        {linear_tc_kernel<2, 0>, linear_tc_kernel<2, 1>, linear_tc_kernel<2, 2>, linear_tc_kernel<2, 3>},
        {linear_tc_kernel<1, 0>, linear_tc_kernel<1, 1>, linear_tc_kernel<1, 2>, linear_tc_kernel<1, 3>}};
    TcKernel kernel = table[BN <= 32 ? 0 : BN <= 64 ? 1 : 2][fi];
    if (prm.ksplit > 1) {
        // a cluster of `ksplit` blocks with this much shared memory must fit the device (it does on a full B200; a
        // partitioned one may not, and then K is not split): checked once per device and cluster size
        static int cluster_ok[kTcMaxSplit + 1][64] = {};
        const int fits = device_once(cluster_ok[prm.ksplit], [&] {
            int n_clusters = 0;
            const cudaError_t e = cudaOccupancyMaxActiveClusters(&n_clusters, kernel, &cfg);
            return (e == cudaSuccess && n_clusters > 0) ? 1 : -1;
        });
        if (fits < 0) {      // fall back to one block per tile
            prm.ksplit = 1;
            cfg.gridDim.z = 1;
            cfg.numAttrs = 1;
        }
    }
    return cuda_status(cudaLaunchKernelEx(&cfg, kernel, prm, code_map));
}

// Failure-path check for the tensor-core kernel's wait helper: a barrier nothing arrives at, no copy or MMA in flight.
__global__ void tc_wait_selftest_kernel(uint32_t limit, int* result) {
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_flag;
    const uint32_t b = (uint32_t)__cvta_generic_to_shared(&bar);
    if (threadIdx.x == 0) { t_mbar_init(b, 1); abort_flag = 0; }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();
    uint32_t bad = 0;
    bad |= t_wait(b, 0, limit) ^ 1u;          // runs out
    bad |= t_wait(b, 0, t_limit(bad)) ^ 1u;   // a later wait of the same role polls once
    t_report(bad, &abort_flag);
    __syncthreads();
    if (threadIdx.x == 0) result[0] = bad ? 0 : 1;
}

int launch_tc_wait_selftest(uint32_t limit, int* result, cudaStream_t st) {
    tc_wait_selftest_kernel<<<1, 32, 0, st>>>(limit, result);
    return cuda_status(cudaGetLastError());
}

int read_tc_status(int clear) {
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_tc_status, sizeof(int)) != cudaSuccess) return HIGGS_ERR_CUDA;
    if (clear && v != 0) {
        const int zero = 0;
        if (cudaMemcpyToSymbol(g_tc_status, &zero, sizeof(int)) != cudaSuccess) return HIGGS_ERR_CUDA;
    }
    return v;
}

}  // namespace higgs
