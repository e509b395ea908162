// Kernel (d), second form: the ternary x int8 GEMM for many tokens with the WEIGHTS in tensor memory.
//
// The first form (prefill_gemm.cu) writes every expanded weight tile to shared memory and the tensor core
// reads it back from there, and the bandwidth of shared memory bounds it.  Here the operands trade places:
// a CTA tile is 128 output features x NTOK tokens, the expanded weights are the A operand of tcgen05.mma
// and live in TENSOR memory (lane = feature, four consecutive k per 32-bit column), the int8 activations
// are the B operand in shared memory.  Per 128-wide k block:
//   producer warp  : TMA loads the activation tile (NTOK x 128 B, 128-byte swizzle) and the packed 2-bit
//                    weight tiles (2 row blocks x 2 column tiles x 1 KiB);
//   expander warps : read the packed tiles once (16 bytes per lane, consecutive), hand every lane the words
//                    of ITS feature with warp shuffles, turn the 2-bit codes into bytes with one mask per four
//                    weights (the field of row 16 f + r stays where it is: the byte is code * 4^f) and write
//                    them to tensor memory with tcgen05.st -- the expanded weights never touch shared memory;
//   MMA warp       : one thread issues four tcgen05.mma kind::i8 (128 x NTOK x 32, u8 weights from tensor
//                    memory x s8 activations from shared memory); tcgen05.commit releases the stage;
//   epilogue warps : tcgen05.ld the int32 sums (lane = feature, column = token), undo 4^f with an exact
//                    shift, subtract the token's sum of q (codes are T + 1), scale by gamma * beta_t / 127,
//                    round to bf16 and store.
// Tensor memory (512 columns): the accumulators (NTOK columns each; two of them when they fit, so that the
// epilogue of a tile overlaps the next tile's MMAs) and a ring of weight k blocks (32 columns each).
// A feature's TMEM lane: quarter q = 2 j + h of the 128 lanes holds, in lane 8 f + g of the quarter, row
// 64 j + 16 f + 8 h + g of the tile -- the order in which the packed layout hands the rows out.
// The kernel is a programmatic dependent of the activation quantiser.  All waits are bounded; on expiry the
// CTA sets the workspace status to BITLINEAR_ERR_TIMEOUT, every role leaves its loop, tensor memory is
// released and the kernel returns.
//
// Roofline: int8 tensor throughput; algorithmic work 2*M*N*K integer operations (Section 2, Eq. 1-3 fix
// the operands; Section 3 "Energy": the matmul dominates).
#include <cuda.h>

#include "internal.cuh"
#include "ptx.cuh"
#include "tma_host.cuh"

namespace bitlinear {

namespace {

using namespace ptx;

constexpr int BW = 128;         // output features per tile (MMA M, TMEM lanes)
constexpr int BK = 128;         // int8 elements (= bytes) of K per stage
constexpr int kACols = BK / 4;  // TMEM columns of one weight k block
constexpr int kTmemCols = 512;
constexpr int kMaxStages = 12;

constexpr int kProducerWarp = 0;
constexpr int kMmaWarp = 1;
// warps 2..5 are the epilogue (one per TMEM lane quarter)
constexpr int kFirstExpanderWarp = 6; // 8 warps: two per lane quarter, taking k blocks in turn
constexpr int kExpanderWarps = 8;
constexpr int kThreads = (kFirstExpanderWarp + kExpanderWarps) * 32; // 448

constexpr uint32_t kPBytes = (BW / kTileRows) * (BK / kTileCols) * kTileBytes; // 4 KiB packed weights

template <int NTOK>
struct Cfg {
    static constexpr int kAccBufs = (2 * NTOK + 4 * kACols <= kTmemCols) ? 2 : 1;
    static constexpr int kRingCols = kTmemCols - kAccBufs * NTOK;
    static constexpr int kSmemStages = (227 * 1024 - 2048) / (NTOK * BK + (int)kPBytes);
    static constexpr int kTmemStages = (kRingCols / kACols < kMaxStages) ? kRingCols / kACols : kMaxStages;
    static constexpr int kStages = kTmemStages < kSmemStages ? kTmemStages : kSmemStages;
    static constexpr uint32_t kXBytes = NTOK * BK; // int8 activations
    static constexpr uint32_t kStageBytes = kXBytes + kPBytes;
    static constexpr uint32_t kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 512 /*barriers*/;
    static_assert(NTOK % 16 == 0 && NTOK >= 16 && NTOK <= 256, "MMA N");
    static_assert(kXBytes % 1024 == 0, "swizzled tiles need 1024-byte alignment");
    static_assert(kStages >= 2, "ring too short");
    static_assert(kSmemBytes <= 232448, "exceeds the 227 KiB shared memory of an SM");
};

struct Barriers {
    uint64_t full[kMaxStages];     // TMA bytes landed (activations + packed weights)
    uint64_t expanded[kMaxStages]; // the weight k block stands in tensor memory
    uint64_t empty[kMaxStages];    // MMAs that read the stage (shared and tensor memory) have completed
    uint64_t acc_full[2];          // accumulator complete
    uint64_t acc_empty[2];         // accumulator drained by the epilogue
    uint32_t tmem_base;
    int abort_flag;
};
static_assert(sizeof(Barriers) <= 512, "barrier block");

struct Params {
    const float *gamma;
    const float *beta;
    const int32_t *rowsum;
    void *out;
    int M, N, KB; // KB = k blocks of 128 columns
    int tiles_t, tiles_w; // token tiles, feature tiles
    int out_i32;
    int32_t *status;
};

template <int NTOK>
__global__ void __launch_bounds__(kThreads, 1)
prefill_ts_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                  const Params p)
{
    using C = Cfg<NTOK>;
    constexpr int kStages = C::kStages, kAccBufs = C::kAccBufs;
    constexpr uint32_t kStageBytes = C::kStageBytes, kXBytes = C::kXBytes;
    constexpr uint32_t kRingCol0 = kAccBufs * NTOK; // first TMEM column of the weight ring

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - raw);
    // layout: [stage][X | P], then the barrier block
    Barriers *bars = reinterpret_cast<Barriers *>(smem + kStages * kStageBytes);
    volatile int *abort_flag = &bars->abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&bars->full[s]), 1);
            mbar_init(smem_u32(&bars->expanded[s]), 4);
            mbar_init(smem_u32(&bars->empty[s]), 1);
        }
        for (int b = 0; b < kAccBufs; ++b) {
            mbar_init(smem_u32(&bars->acc_full[b]), 1);
            mbar_init(smem_u32(&bars->acc_empty[b]), 4);
        }
        bars->abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == kMmaWarp) {
        tmem_alloc(smem_u32(&bars->tmem_base), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;

    const int n_tiles = p.tiles_t * p.tiles_w;
    const int KB = p.KB;

    if (warp == kProducerWarp) {
        if (lane == 0) {
            prefetch_tensormap(&tmap_x);
            prefetch_tensormap(&tmap_w);
            griddep_wait(); // the activations are written by the launch before this one
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
                const int m0 = (tile % p.tiles_t) * NTOK;
                const int n0 = (tile / p.tiles_t) * BW;
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = it % kStages;
                    const uint32_t round = it / kStages;
                    if (round > 0 && !mbar_wait_bounded(smem_u32(&bars->empty[s]), (round - 1) & 1, abort_flag)) {
                        ok = false;
                        break;
                    }
                    const uint32_t full = smem_u32(&bars->full[s]);
                    const uint32_t x_dst = base + s * kStageBytes;
                    mbar_arrive_expect_tx(full, kXBytes + kPBytes);
                    tma_load_2d(x_dst, &tmap_x, kb * BK, m0, full); // x = byte column (multiple of 128)
                    tma_load_3d(x_dst + kXBytes, &tmap_w, 0, kb * (BK / kTileCols), n0 / kTileRows, full); // whole tiles
                }
            }
        }
    } else if (warp == kMmaWarp) {
        constexpr uint32_t idesc = idesc_i8(BW, NTOK, /*a_signed=*/0, /*b_signed=*/1);
        uint32_t it = 0, tile_it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++tile_it) {
            const int buf = tile_it % kAccBufs;
            const uint32_t use = tile_it / kAccBufs;
            if (use > 0 && !mbar_wait_bounded(smem_u32(&bars->acc_empty[buf]), (use - 1) & 1, abort_flag)) break;
            tc_fence_after_sync();
            const uint32_t d_tmem = tmem_base + (uint32_t)(buf * NTOK);
            for (int kb = 0; kb < KB; ++kb, ++it) {
                const int s = it % kStages;
                const uint32_t parity = (it / kStages) & 1;
                if (!mbar_wait_bounded(smem_u32(&bars->full[s]), parity, abort_flag) ||
                    !mbar_wait_bounded(smem_u32(&bars->expanded[s]), parity, abort_flag)) {
                    ok = false;
                    break;
                }
                tc_fence_after_sync();
                if (lane == 0) {
                    const uint32_t x_addr = base + s * kStageBytes;
                    const uint32_t a_tmem = tmem_base + kRingCol0 + (uint32_t)(s * kACols);
#pragma unroll
                    for (int k4 = 0; k4 < BK / 32; ++k4) {
                        mma_i8_ts(d_tmem, a_tmem + 8 * k4, smem_desc_k_sw128(x_addr + 32 * k4), idesc,
                                  (kb > 0 || k4 > 0) ? 1u : 0u);
                    }
                    mma_commit(smem_u32(&bars->empty[s])); // stage reusable once these MMAs have read it
                }
                __syncwarp();
            }
            if (ok && lane == 0) mma_commit(smem_u32(&bars->acc_full[buf]));
            __syncwarp();
        }
    } else if (warp >= kFirstExpanderWarp) {
        // This warp writes TMEM lane quarter q = warp % 4: rows 16 f + 8 h + g (f = 0..3, g = 0..7) of row block
        // j of the tile, j = q / 2, h = q % 2; lane 8 f + g takes row (f, g).  Of the packed tile (row block j,
        // column tile kti) lane L loads the 16 bytes at slot L of each slab s: the codes of rows 16 f' + 8 h' + g'
        // (g' = L / 4) at columns 16 tq' + 8 s + 4 hi + b (tq' = L % 4; word 2 hi + h', byte b, field f').  So
        // the four bytes of this lane's row at columns 16 tq + 8 s + 4 hi + (0..3) are word 2 hi + h of lane
        // 4 g + tq, masked to field f: TMEM column (64 kti + 16 tq + 8 s + 4 hi) / 4 of the k block.
        const int ew = warp - kFirstExpanderWarp;
        const int q = warp & 3, turn = ew >> 2;
        const int j = q >> 1, h = q & 1;
        const int g = lane & 7, f = lane >> 3;
        const uint32_t mask = 0x03030303u << (2 * f);
        uint32_t it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
            for (int kb = 0; kb < KB; ++kb, ++it) {
                if ((int)(it & 1u) != turn) continue;
                const int s = it % kStages;
                const uint32_t parity = (it / kStages) & 1;
                if (!mbar_wait_bounded(smem_u32(&bars->full[s]), parity, abort_flag)) {
                    ok = false;
                    break;
                }
                const uint8_t *packed = smem + s * kStageBytes + kXBytes + (size_t)(j * (BK / kTileCols)) * kTileBytes;
                uint32_t sel[2][2][2]; // [kti][s][hi]: the word 2 hi + h of this lane's 16 bytes
#pragma unroll
                for (int kti = 0; kti < 2; ++kti) {
#pragma unroll
                    for (int sl = 0; sl < 2; ++sl) {
                        const uint4 w = *reinterpret_cast<const uint4 *>(packed + kti * kTileBytes + sl * 512 + lane * 16);
                        sel[kti][sl][0] = h ? w.y : w.x;
                        sel[kti][sl][1] = h ? w.w : w.z;
                    }
                }
                uint32_t r[kACols];
#pragma unroll
                for (int kti = 0; kti < 2; ++kti) {
#pragma unroll
                    for (int tq = 0; tq < 4; ++tq) {
#pragma unroll
                        for (int sl = 0; sl < 2; ++sl) {
#pragma unroll
                            for (int hi = 0; hi < 2; ++hi)
                                r[16 * kti + 4 * tq + 2 * sl + hi] =
                                    __shfl_sync(0xffffffffu, sel[kti][sl][hi], 4 * g + tq) & mask;
                        }
                    }
                }
                tc_fence_after_sync(); // the MMAs that read this ring slot completed before the stage was refilled
                tmem_st_32x32(tmem_base + ((uint32_t)(32 * q) << 16) + kRingCol0 + (uint32_t)(s * kACols), r);
                tmem_st_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars->expanded[s]));
            }
        }
    } else {
        // epilogue: warp w may touch TMEM lanes 32*(w % 4) .. +31; this thread's lane holds one feature
        const int q = warp & 3;
        const int f = lane >> 3;
        const int row = 64 * (q >> 1) + 16 * f + 8 * (q & 1) + (lane & 7);
        uint32_t tile_it = 0;
        const float gamma = p.out_i32 ? 0.0f : *p.gamma;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++tile_it) {
            const int m0 = (tile % p.tiles_t) * NTOK;
            const int n = (tile / p.tiles_t) * BW + row;
            const int buf = tile_it % kAccBufs;
            const uint32_t parity = (tile_it / kAccBufs) & 1;
            const bool n_ok = n < p.N;
            if (!mbar_wait_bounded(smem_u32(&bars->acc_full[buf]), parity, abort_flag)) break;
            tc_fence_after_sync();
#pragma unroll 1
            for (int c = 0; c < NTOK / 32; ++c) {
                const int t0 = m0 + 32 * c;
                if (t0 >= p.M) break; // (the same for the whole warp)
                // lane i keeps the sum of q and the scale of token t0 + i
                int my_rowsum = 0;
                float my_scale = 0.0f;
                if (t0 + lane < p.M) {
                    my_rowsum = p.rowsum[t0 + lane];
                    if (!p.out_i32) my_scale = __fdiv_rn(__fmul_rn(gamma, p.beta[t0 + lane]), (float)kQb);
                }
                uint32_t v[32];
                tmem_ld_32x32(tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(buf * NTOK + c * 32), v);
                tmem_ld_wait();
                const int n_tok = min(32, p.M - t0);
                if (p.out_i32) {
                    int32_t *dst = reinterpret_cast<int32_t *>(p.out) + (size_t)t0 * p.N + n;
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int rs = __shfl_sync(0xffffffffu, my_rowsum, i);
                        if (i < n_tok && n_ok) dst[(size_t)i * p.N] = ((int)v[i] >> (2 * f)) - rs;
                    }
                } else {
                    __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(p.out) + (size_t)t0 * p.N + n;
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int rs = __shfl_sync(0xffffffffu, my_rowsum, i);
                        const float sc = __shfl_sync(0xffffffffu, my_scale, i);
                        if (i < n_tok && n_ok)
                            dst[(size_t)i * p.N] = __float2bfloat16_rn(__fmul_rn((float)(((int)v[i] >> (2 * f)) - rs), sc));
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bars->acc_empty[buf]));
        }
    }

    // common tail: every thread arrives here, also after an expired wait
    if (*abort_flag) {
        if (threadIdx.x == 0) atomicExch(p.status, (int32_t)BITLINEAR_ERR_TIMEOUT);
        // give copies and MMAs that may still be in flight time to land before shared memory and TMEM go away
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == kMmaWarp) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ---- host side ---------------------------------------------------------------------------------

template <int NTOK>
cudaError_t launch_ts(const void *packed, const float *gamma, const int8_t *Xq, const float *beta,
                      const int32_t *rowsum, int64_t M, int64_t K, int64_t N, void *out, int out_i32,
                      WorkspaceHeader *hdr, cudaStream_t stream)
{
    if (!encode_tiled_fn()) return cudaErrorNotSupported;
    const int KB = (int)((K + BK - 1) / BK);

    // activations: box of NTOK rows; weights: box of 2 row blocks x 2 column tiles
    CUtensorMap tmap_x, tmap_w;
    if (!encode_activation_map(&tmap_x, Xq, M, K, NTOK) || !encode_packed_weight_map(&tmap_w, packed, N, K, BW / kTileRows))
        return cudaErrorInvalidValue;

    Params p;
    p.gamma = gamma;
    p.beta = beta;
    p.rowsum = rowsum;
    p.out = out;
    p.M = (int)M;
    p.N = (int)N;
    p.KB = KB;
    p.tiles_t = (int)((M + NTOK - 1) / NTOK);
    p.tiles_w = (int)((N + BW - 1) / BW);
    p.out_i32 = out_i32;
    p.status = &hdr->status;

    static bool attr_set[64] = {false};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(prefill_ts_kernel<NTOK>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)Cfg<NTOK>::kSmemBytes);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    int grid = p.tiles_t * p.tiles_w;
    if (grid > sm_count()) grid = sm_count();
    // programmatic dependent launch: see the head of this file
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = Cfg<NTOK>::kSmemBytes;
    cfg.stream = stream;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    void *args[] = {(void *)&tmap_x, (void *)&tmap_w, (void *)&p};
    return cudaLaunchKernelExC(&cfg, (const void *)prefill_ts_kernel<NTOK>, args);
}

} // namespace

cudaError_t launch_prefill_ts(const void *packed, const float *gamma, const int8_t *Xq, const float *beta,
                              const int32_t *rowsum, int64_t M, int64_t K, int64_t N, void *out, int out_i32,
                              int tokens_per_tile, WorkspaceHeader *hdr, cudaStream_t stream)
{
    if (tokens_per_tile == 64)
        return launch_ts<64>(packed, gamma, Xq, beta, rowsum, M, K, N, out, out_i32, hdr, stream);
    if (tokens_per_tile == 192)
        return launch_ts<192>(packed, gamma, Xq, beta, rowsum, M, K, N, out, out_i32, hdr, stream);
    return launch_ts<256>(packed, gamma, Xq, beta, rowsum, M, K, N, out, out_i32, hdr, stream);
}

} // namespace bitlinear
