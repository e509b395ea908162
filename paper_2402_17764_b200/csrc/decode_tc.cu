// Kernel (c'), 17 to 64 tokens: the ternary x int8 matmul with the WEIGHTS as the stationary 128-row operand of the
// tcgen05 tensor cores and the tokens as the MMA's N.
//
// With a few dozen tokens the matmul (Section 1: integer additions; the weights' way from DRAM is the cost) is still a
// stream of weights, and what limits a tensor-core kernel is everything around the MMAs.  In the GEMM of
// prefill_gemm.cu the tokens are the 128-row operand: with 64 tokens an MMA runs half empty, and the expanded weights
// (four times the packed bytes) go through shared memory twice, written by the expander and read by the tensor core.
// Here a CTA tile is 256 features x 64 tokens, per 128-wide k block:
//   producer threads: four, each every fourth k block (an issued copy costs its thread 100 to 150 cycles): TMA loads 64
//                     rows of int8 activations (128-byte swizzle, the MMA's B operand) and 8 KiB of packed weights (four
//                     row blocks x two column tiles, 128-byte swizzle) into a ring of stages;
//   expander warps  : sixteen, one per (lane quarter of tensor memory, feature block, parity of the k block): every thread
//                     loads ONE 16-byte piece of packed words per MMA k step, keeps the fields of four output rows with one mask
//                     each (the byte is code * 4^f) and writes them with tcgen05.st.16x256b straight into TENSOR memory
//                     as the A operand of the MMAs (lane = output row, 32 columns = the k block): the expanded weights
//                     never touch shared memory, and no packed byte is fetched twice by a warp (store_unit below);
//   MMA threads     : four, one per (feature block of 128, parity of the k block), because one thread issues a
//                     tcgen05.mma only every 110 cycles whatever its size, and an MMA of 128 x 64 x 32 takes 36: each
//                     issues the four MMAs of its k blocks (A from tensor memory, B from the stage) and commits to the
//                     barrier that frees the unit of the A ring (the MMAs' N is 32, 48 or 64: the largest M of the launch
//                     rounded up to 16).  The two threads of a feature block add into the SAME
//                     accumulator, which the epilogue left zeroed, so that no MMA has to be the first (measured on
//                     B200: sums of MMAs issued by four threads into one accumulator are exact);
//   epilogue warps  : four: tcgen05.ld the finished sums (lane = feature, column = token), undo the 4^f of their row
//                     with an exact shift, subtract the token's sum of q (codes are T + 1), scale by
//                     gamma * beta_t / Q_b, round to bf16, store, and write zeros back, while the MMAs fill the other
//                     pair of accumulators.
// Which output row stands in which lane is free (the epilogue undoes it): lane 32 q + l of feature block fb holds row
// 128 fb + 64 (q / 2) + 16 (l / 8) + 8 (q % 2) + g of the tile, g = (l % 8) / 2 + 4 (l % 2): the 8 h (q % 2) of the
// packed layout is the same for a whole warp (which two of the four words of a piece it keeps is fixed at compile
// time), the field f = l / 8 is the lane eighth the 16x256b store addresses, and the order of g within eight lanes
// keeps the loads of a quarter-warp in eight different bank groups.
// All waits are bounded; on expiry the CTA sets the workspace status to BITLINEAR_ERR_TIMEOUT, every role leaves its
// loop, tensor memory is released and the kernel returns.
//
// Roofline: HBM (0.25 bytes per weight); the tensor pipe is about 40 % busy at 64 tokens.
#include <cuda.h>

#include "gemm_problem.cuh"
#include "internal.cuh"
#include "ptx.cuh"

namespace bitlinear {

namespace {

using namespace ptx;

constexpr int kTokens = 64;        // MMA N: rows of activations per stage (rows past M read zero)
constexpr int kFeatureBlocks = 2;  // of 128 features per CTA tile
constexpr int kASlots = 4;         // k blocks whose A operands stand in tensor memory
constexpr int kAUnits = kASlots * kFeatureBlocks;
constexpr int kAccCols = kTokens;  // columns of one accumulator
constexpr uint32_t kAColumn0 = 2 * kFeatureBlocks * kAccCols; // accumulators: two buffers x feature blocks, then the A units
constexpr uint32_t kTmemCols = 512;
static_assert(kAColumn0 + kAUnits * 32 <= kTmemCols, "tensor memory");

constexpr int kProducerWarps = 4;      // one issuing thread each: k blocks it % 4 (an issued copy costs its thread 100 to 150 cycles)
constexpr int kFirstMmaWarp = 4;       // 4 warps, one issuing thread each: feature block x parity of the k block
constexpr int kFirstEpilogueWarp = 8;  // 4 warps
constexpr int kFirstExpanderWarp = 12; // 16 warps: lane quarter x slot of the A ring
constexpr int kExpanderWarps = 16;
constexpr int kThreads = (kFirstExpanderWarp + kExpanderWarps) * 32; // 896

constexpr uint32_t kActBytes = kTokens * BK;   // 8 KiB
constexpr uint32_t kPackedBytes = 8192;        // 4 row blocks x 2 column tiles
constexpr uint32_t kStageBytes = kActBytes + kPackedBytes;
constexpr int kMaxStages = 13;
constexpr uint32_t kSmemLimit = 232448; // 227 KiB
constexpr uint32_t kLongPauseNs = 400;  // between the polls of the roles that wait long and are not on the critical path

struct Barriers {
    uint64_t full[kMaxStages];        // TMA bytes landed (activations + packed weights)
    uint64_t stage_empty[kMaxStages]; // the MMAs of both feature blocks have read the stage (passed on by an expander warp)
    uint64_t a_full[kAUnits];         // A operand of (slot, feature block) written (four lane quarters)
    uint64_t a_empty[kAUnits];        // the MMAs that read it have completed
    uint64_t acc_full[2];             // accumulators of a tile complete (four MMA threads)
    uint64_t acc_empty[2];            // drained and zeroed (four epilogue warps)
    uint32_t tmem_base;
    int abort_flag;
    float scale[4][kTokens];          // per epilogue warp: gamma * beta_t / Q_b and the sum of q of every token
    int rowsum[4][kTokens];
};
constexpr uint32_t kBarrierBytes = 2560;
static_assert(sizeof(Barriers) <= kBarrierBytes, "barrier block");

inline int stages_that_fit()
{
    const int n = (int)((kSmemLimit - 1024 - kBarrierBytes) / kStageBytes);
    return n < kMaxStages ? n : kMaxStages;
}
inline uint32_t smem_bytes_for(int n_stages) { return 1024 + (uint32_t)n_stages * kStageBytes + kBarrierBytes; }

// One A unit = the 32 rows of a lane quarter x one k block, written with tcgen05.st.16x256b: in that shape thread
// 4 j + kq of the warp holds, for each of the four MMA k steps, columns 2 kq and 2 kq + 1 (eight consecutive bytes of K)
// of lanes j and j + 8 of a 16-lane half.  Those eight bytes of K are exactly one 16-byte piece of the packed layout: the
// piece (slab s, slot 4 g + tq) holds, as words 2 hi + h, the codes of rows 16 f + 8 h + g at columns
// 16 tq + 8 s + 4 hi + b, so thread (j, kq) loads ONE piece per k step -- (column tile k4 / 2, tq = 2 (k4 % 2) + kq / 2,
// s = kq % 2) of its row group g -- keeps the two words of the warp's h, and the four masks give the bytes code * 4^f
// of the four rows f: lanes j and j + 8 of the lower half (f = 0, 1) and of the upper half (f = 2, 3).  Every lane of a
// load reads a different piece (32 x 16 bytes per instruction, nothing fetched twice), and with g = j / 2 + 4 (j % 2) the
// eight lanes of a quarter-warp fall into eight different bank groups of the swizzled stage.
__device__ __forceinline__ void tmem_st_16x256_x4(uint32_t taddr, const uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.16x256b.x4.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
        "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}

// the eight words of this thread for one unit: [k step][hi]; `w`: the thread's base inside the packed part of the stage
// (row block, 512 s, 128 (g / 2), 64 ((g % 2) ^ s) applied); off_e[e] = 16 ((2 e + kq / 2) ^ (g / 2))
template <int H>
__device__ __forceinline__ void load_unit(uint32_t (&x)[4][2], const uint8_t *w, const uint32_t (&off_e)[2])
{
#pragma unroll
    for (int k4 = 0; k4 < 4; ++k4) {
        const uint4 v = *reinterpret_cast<const uint4 *>(w + (k4 >> 1) * kTileBytes + off_e[k4 & 1]);
        x[k4][0] = H ? v.y : v.x;
        x[k4][1] = H ? v.w : v.z;
    }
}

// masks and stores them: `taddr` = lane quarter base + first column of the unit
__device__ __forceinline__ void store_unit(const uint32_t (&x)[4][2], uint32_t taddr)
{
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) { // lanes 16 hh .. 16 hh + 15: rows f = 2 hh (lanes j) and 2 hh + 1 (lanes j + 8)
        uint32_t r[16];
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const uint32_t mask = 0x03030303u << (2 * (2 * hh + e));
                r[4 * k4 + 2 * e] = x[k4][0] & mask;
                r[4 * k4 + 2 * e + 1] = x[k4][1] & mask;
            }
        }
        tmem_st_16x256_x4(taddr + ((uint32_t)(16 * hh) << 16), r);
    }
}

template <bool kTable>
__global__ void __launch_bounds__(kThreads, 1)
decode_tc_kernel(const __grid_constant__ GemmProblem one, const GemmProblem *__restrict__ table, int n_problems, int n_tiles,
                 int n_stages, int mma_n, const WaitHooks hooks)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u; // swizzled tiles need 1024-byte alignment
    uint8_t *smem = smem_raw + (base - raw);
    Barriers *bars = reinterpret_cast<Barriers *>(smem + (uint32_t)n_stages * kStageBytes);
    volatile int *abort_flag = &bars->abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int q = warp & 3; // the lane quarter of tensor memory this warp may touch

    if (threadIdx.x == 0) {
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(smem_u32(&bars->full[s]), 1);
            mbar_init(smem_u32(&bars->stage_empty[s]), kFeatureBlocks);
        }
        for (int u = 0; u < kAUnits; ++u) {
            mbar_init(smem_u32(&bars->a_full[u]), 4);
            mbar_init(smem_u32(&bars->a_empty[u]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bars->acc_full[b]), 4);
            mbar_init(smem_u32(&bars->acc_empty[b]), 4);
        }
        bars->abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == kFirstMmaWarp) {
        tmem_alloc(smem_u32(&bars->tmem_base), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(32 * q) << 16);
    if (warp >= kFirstEpilogueWarp && warp < kFirstExpanderWarp) {
        // every MMA accumulates: the accumulators start as zeros, and the epilogue leaves them so
        uint32_t z[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) z[i] = 0u;
#pragma unroll
        for (uint32_t c = 0; c < kAColumn0; c += 16) tmem_st_32x16(lane_addr + c, z);
        tmem_st_wait();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();

    int32_t *const status = kTable ? table[0].p.status : one.p.status; // (the same for every matmul of a launch)

    if (warp < kProducerWarps) {
        if (lane == 0) {
            ProblemCursor<kTable> cur(one, table, n_problems);
            if (!kTable) {
                prefetch_tensormap(&one.tmap_x);
                prefetch_tensormap(&one.tmap_w);
            }
            griddep_wait(); // the activations are written by the launch before this one
            int s = 0;
            uint32_t round = 0, it = 0;
            bool ok = true;
            for (int tile = (int)blockIdx.x; ok && tile < n_tiles; tile += (int)gridDim.x) {
                const GemmProblem &g = cur.seek(tile);
                const int n0 = (tile - g.p.tile_begin) * BN;
                const int KB = g.p.KB; // (a copy: the table stands in global memory, and the loop's asm statements clobber memory)
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    if ((it & (kProducerWarps - 1)) == (uint32_t)warp) {
                        if (round > 0 &&
                            !mbar_wait_bounded(smem_u32(&bars->stage_empty[s]), (round - 1) & 1, abort_flag, hooks.limit_us, kLongPauseNs)) {
                            ok = false;
                            break;
                        }
                        // (test device: the first CTA leaves out the arrival that announces its first stage's bytes, and
                        // the loads it announces with it, so that nothing is in flight for a phase that never completes)
                        if (!(hooks.skip_arrive && blockIdx.x == 0 && it == 0)) {
                            const uint32_t full = smem_u32(&bars->full[s]);
                            const uint32_t dst = base + (uint32_t)s * kStageBytes;
                            mbar_arrive_expect_tx(full, kStageBytes);
                            tma_load_2d(dst, &g.tmap_x, kb * BK, 0, full);
                            tma_load_3d(dst + kActBytes, &g.tmap_w, 0, kb * 16, n0 / kTileRows, full);
                        }
                    }
                    if (++s == n_stages) {
                        s = 0;
                        ++round;
                    }
                }
            }
        }
    } else if (warp < kFirstEpilogueWarp) {
        // MMA thread j: feature block j % 2, the k blocks (counted over all tiles of this CTA) of parity j / 2
        if (lane == 0) {
            const int j = warp - kFirstMmaWarp;
            const int fb = j & 1;
            const uint32_t par = (uint32_t)(j >> 1);
            const uint32_t idesc = idesc_i8(128, mma_n, /*a_signed=*/0, /*b_signed=*/1); // (fewer tokens: narrower, shorter MMAs)
            const uint32_t desc_hi = (uint32_t)(smem_desc_k_sw128(0) >> 32);
            const uint32_t b_lo0 = (uint32_t)smem_desc_k_sw128(base);
            ProblemCursor<kTable> cur(one, table, n_problems);
            uint32_t it = 0, tile_it = 0;
            int s = 0;
            bool ok = true;
            for (int tile = (int)blockIdx.x; ok && tile < n_tiles; tile += (int)gridDim.x, ++tile_it) {
                const int KB = cur.seek(tile).p.KB;
                const uint32_t buf = tile_it & 1u, use = tile_it >> 1;
                if (use > 0 && !mbar_wait_bounded(smem_u32(&bars->acc_empty[buf]), (use - 1) & 1, abort_flag, hooks.limit_us)) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + (buf * kFeatureBlocks + (uint32_t)fb) * kAccCols;
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    if ((it & 1u) == par) {
                        const uint32_t unit = (it & (kASlots - 1)) * kFeatureBlocks + (uint32_t)fb;
                        if (!mbar_wait_bounded(smem_u32(&bars->a_full[unit]), (it / kASlots) & 1, abort_flag, hooks.limit_us)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after_sync();
                        const uint32_t a_tmem = tmem_base + kAColumn0 + unit * 32u;
                        const uint32_t b_lo = b_lo0 + (((uint32_t)s * kStageBytes) >> 4);
#pragma unroll
                        for (int k4 = 0; k4 < BK / 32; ++k4) // 32 bytes of K: 8 columns of A, 2 descriptor units of B
                            mma_i8_ts(d_tmem, a_tmem + 8u * k4, ((uint64_t)desc_hi << 32) | (b_lo + 2u * k4), idesc, 1u);
                        mma_commit(smem_u32(&bars->a_empty[unit])); // (one commit: it costs the thread as much as an MMA)
                    }
                    if (++s == n_stages) s = 0;
                }
                if (ok) mma_commit(smem_u32(&bars->acc_full[buf]));
            }
        }
    } else if (warp >= kFirstExpanderWarp) {
        // Expander warp (lane quarter q, feature block fb, parity par): its 32 rows of feature block fb in the k blocks of
        // parity par, i.e. in slots par and par + 2 of the A ring in turn.  Every (slot, feature block) unit has barriers
        // of its own, so that the MMAs of one feature block never wait for the expansion of the other.  The packed words
        // are loaded before the warp waits for the unit to be free: only the masks, the stores and their wait stand
        // between the MMAs that free a unit and the MMAs that use it next.  Those MMAs, of the k block four back, have
        // completed once `a_empty` lets the warp pass: the warps of quarter 0 hand that k block's stage back to the
        // producer (one arrival per feature block), which spares the MMA threads a second commit.
        const int e = (warp - kFirstExpanderWarp) >> 2; // (warp % 4 is the lane quarter)
        const int fb = e & 1;
        const uint32_t par = (uint32_t)(e >> 1);
        const int j = lane >> 2, kq = lane & 3, h = q & 1, t = q >> 1;
        const int g8 = (j >> 1) + 4 * (j & 1), sl = kq & 1;
        const uint32_t lane_off = kActBytes + (uint32_t)((2 * fb + t) * 2 * kTileBytes) + 512u * (uint32_t)sl + 128u * (uint32_t)(g8 >> 1) +
                                  64u * (uint32_t)((g8 & 1) ^ sl);
        const uint32_t off_e[2] = {16u * (uint32_t)((kq >> 1) ^ (g8 >> 1)), 16u * (uint32_t)((2 + (kq >> 1)) ^ (g8 >> 1))};
        ProblemCursor<kTable> cur(one, table, n_problems);
        uint32_t it = 0, round = 0;
        int s = 0, s_two_back = 0, s_four_back = 0; // stages of this k block and of this warp's last two
        bool ok = true;
        for (int tile = (int)blockIdx.x; ok && tile < n_tiles; tile += (int)gridDim.x) {
            const int KB = cur.seek(tile).p.KB;
            for (int kb = 0; kb < KB; ++kb, ++it) {
                if ((it & 1u) == par) {
                    const uint32_t unit = (it & (kASlots - 1)) * kFeatureBlocks + (uint32_t)fb;
                    const uint32_t a_use = it / kASlots;
                    if (!mbar_wait_bounded(smem_u32(&bars->full[s]), round & 1, abort_flag, hooks.limit_us)) {
                        ok = false;
                        break;
                    }
                    uint32_t x[4][2];
                    if (h)
                        load_unit<1>(x, smem + (uint32_t)s * kStageBytes + lane_off, off_e);
                    else
                        load_unit<0>(x, smem + (uint32_t)s * kStageBytes + lane_off, off_e);
                    if (a_use > 0 && !mbar_wait_bounded(smem_u32(&bars->a_empty[unit]), (a_use - 1) & 1, abort_flag, hooks.limit_us)) {
                        ok = false;
                        break;
                    }
                    if (a_use > 0 && q == 0 && lane == 0) mbar_arrive(smem_u32(&bars->stage_empty[s_four_back]));
                    tc_fence_after_sync();
                    store_unit(x, lane_addr + kAColumn0 + unit * 32u);
                    tmem_st_wait();
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bars->a_full[unit]));
                    s_four_back = s_two_back;
                    s_two_back = s;
                }
                if (++s == n_stages) {
                    s = 0;
                    ++round;
                }
            }
        }
    } else {
        // epilogue warp of lane quarter q
        griddep_wait(); // the tokens' scales and sums are written by the launch before this one
        ProblemCursor<kTable> cur(one, table, n_problems);
        float *scale = bars->scale[q];
        int *rowsum = bars->rowsum[q];
        const int shift = 2 * (lane >> 3);
        const int row_in_block = 64 * (q >> 1) + 16 * (lane >> 3) + 8 * (q & 1) + ((lane & 7) >> 1) + 4 * (lane & 1);
        uint32_t tile_it = 0;
        for (int tile = (int)blockIdx.x; tile < n_tiles; tile += (int)gridDim.x, ++tile_it) {
            const Params p = cur.seek(tile).p; // (a copy in registers: the table stands in global memory)
            const int n0 = (tile - p.tile_begin) * BN;
            const uint32_t buf = tile_it & 1u;
            // this warp's copy of the tokens' scales and sums (the other warps may still read theirs of the last tile)
            __syncwarp();
#pragma unroll
            for (int m = lane; m < kTokens; m += 32) {
                int rs = 0;
                float sc = 0.0f;
                if (m < p.M) {
                    rs = p.rowsum[m];
                    if (!p.out_i32) sc = __fdiv_rn(__fmul_rn(*p.gamma, p.beta[m]), p.qb);
                }
                rowsum[m] = rs;
                scale[m] = sc;
            }
            __syncwarp();
            if (!mbar_wait_bounded(smem_u32(&bars->acc_full[buf]), (tile_it >> 1) & 1, abort_flag, hooks.limit_us, kLongPauseNs)) break;
            tc_fence_after_sync();
            uint32_t z[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) z[i] = 0u;
#pragma unroll 1
            for (int fb = 0; fb < kFeatureBlocks; ++fb) {
                const int n = n0 + 128 * fb + row_in_block;
                const uint32_t acc = lane_addr + (buf * kFeatureBlocks + (uint32_t)fb) * kAccCols;
#pragma unroll 1
                for (int half = 0; 32 * half < mma_n; ++half) { // (columns no MMA wrote stay zero)
                    uint32_t v[32];
                    tmem_ld_32x32(acc + 32u * half, v);
                    tmem_ld_wait();
                    tmem_st_32x16(acc + 32u * half, z);
                    tmem_st_32x16(acc + 32u * half + 16u, z);
                    if (n < p.N) {
                        // all results first, then the stores: a store between two loads of the tokens' scales would
                        // order them (the compiler cannot tell the output from the shared arrays) and make every
                        // element wait for the one before it
                        const int count = p.M - 32 * half; // tokens of this half that exist (may be <= 0 or > 32)
#pragma unroll
                        for (int i0 = 0; i0 < 32; i0 += 16) {
                            if (i0 >= count) break; // (the same for the whole warp)
                            if (p.out_i32) {
                                int32_t *dst = reinterpret_cast<int32_t *>(p.out) + (size_t)(32 * half + i0) * p.N + n;
                                int a[16];
#pragma unroll
                                for (int i = 0; i < 16; ++i) a[i] = ((int)v[i0 + i] >> shift) - rowsum[32 * half + i0 + i];
#pragma unroll
                                for (int i = 0; i < 16; ++i)
                                    if (i0 + i < count) dst[(size_t)i * p.N] = a[i];
                            } else {
                                __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(p.out) + (size_t)(32 * half + i0) * p.N + n;
                                __nv_bfloat16 y[16];
#pragma unroll
                                for (int i = 0; i < 16; ++i)
                                    y[i] = __float2bfloat16_rn(
                                        __fmul_rn((float)(((int)v[i0 + i] >> shift) - rowsum[32 * half + i0 + i]), scale[32 * half + i0 + i]));
#pragma unroll
                                for (int i = 0; i < 16; ++i)
                                    if (i0 + i < count) dst[(size_t)i * p.N] = y[i];
                            }
                        }
                    }
                }
            }
            tmem_st_wait();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bars->acc_empty[buf]));
        }
    }

    // common tail: every thread arrives here, also after an expired wait; the flag is looked at AFTER the barrier (a
    // thread whose role ended early gets here long before a wait of another role can expire)
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) { // (the same for every thread now)
        if (threadIdx.x == 0) atomicExch(status, (int32_t)BITLINEAR_ERR_TIMEOUT);
        // give copies and MMAs that may still be in flight time to land before shared memory and TMEM go away
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == kFirstMmaWarp) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

} // namespace


cudaError_t launch_decode_tc(const GemmProblem &one, const GemmProblem *table, int n, int n_tiles, int max_M, cudaStream_t stream)
{
    const void *kernel = table ? (const void *)decode_tc_kernel<true> : (const void *)decode_tc_kernel<false>;
    int n_stages = stages_that_fit();
    const uint32_t smem_bytes = smem_bytes_for(n_stages);
    static bool attr_set[64] = {false};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        for (const void *k : {(const void *)decode_tc_kernel<true>, (const void *)decode_tc_kernel<false>}) {
            cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit);
            if (e != cudaSuccess) return e;
        }
        attr_set[dev] = true;
    }
    if (n_tiles <= 0) return cudaSuccess;
    const int sms = sm_count();
    const int grid = n_tiles < sms ? n_tiles : sms;
    // programmatic dependent launch: set-up (barriers, tensor memory) runs while the quantiser finishes
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    WaitHooks hooks = take_wait_hooks();
    int mma_n = max_M <= 32 ? 32 : (max_M <= 48 ? 48 : kTokens); // columns of the MMAs: the tokens, rounded up to 16
    void *args[] = {(void *)&one, (void *)&table, (void *)&n, (void *)&n_tiles, (void *)&n_stages, (void *)&mma_n, (void *)&hooks};
    return cudaLaunchKernelExC(&cfg, kernel, args);
}

} // namespace bitlinear
