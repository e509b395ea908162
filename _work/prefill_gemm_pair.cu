// Kernel (d), two-SM form: the ternary x int8 GEMM for many tokens with tcgen05.mma.cta_group::2.
//
// The one-SM kernel (prefill_gemm.cu) is limited by shared-memory bandwidth: per 128-wide k block an SM
// reads 48 KB of operands for the MMA, receives 24 KB from TMA and moves 40 KB through the expander, which
// keeps the tensor pipe below 60 %.  Here two CTAs on neighbouring SMs (a cluster of two) work on one tile
// of 256 tokens x 256 output features: each CTA holds its own 128 tokens and only ITS HALF of the weight
// tile (128 features), so per k block an SM expands 4 KB instead of 8 KB of packed weights, receives 20 KB
// instead of 24 KB, and the MMA reads 32 KB instead of 48 KB of its shared memory.  The MMAs are issued by
// one thread of the leader CTA (cluster rank 0) and write the accumulators of both CTAs' tensor memory.
//
// Per CTA: TMA producer warp, MMA warp (leader) / relay warp (peer: tells the leader when the peer's half
// of a stage is ready), 4 epilogue warps, 4 expander warps.  Barriers that both CTAs use:
//   ready_peer[s] (in the leader)  <- peer's relay warp: peer's activations landed and weights expanded
//   empty[s]      (in both)        <- tcgen05.commit (multicast): the MMAs that read stage s are done
//   acc_full[b]   (in both)        <- tcgen05.commit (multicast): accumulator b complete
//   acc_empty[b]  (in the leader)  <- the epilogue warps of both CTAs: accumulator b drained
// All waits are bounded; on expiry a CTA raises its abort flag, its roles leave their loops, the peer runs
// into its own limits, and both meet at the cluster barrier in front of the release of tensor memory.
//
// Measured on B200: bit-exact, but 1.15 POP/s where the one-SM kernel reaches 2.2 POP/s (13824 x 5120, 2048
// tokens).  A register-only issue loop reaches 4.57 POP/s in both forms, so the MMA itself is not the limit;
// with the pipeline around it the leader's MMA issue blocks for ~1150 clocks per k block (one-SM form:
// ~950 for half the work), also with TMA, expander and epilogue switched off one by one.  The cause is not found yet; the library therefore dispatches to the one-SM kernel and
// this one is reachable through BITLINEAR_PATH_TCGEN05_PAIR of the test hook only.
//
// Roofline: int8 tensor throughput; algorithmic work 2*M*N*K integer operations.
#include <cuda.h>

#include "internal.cuh"
#include "ptx.cuh"
#include "tma_host.cuh"

namespace bitlinear {

namespace {

using namespace ptx;

constexpr int BM = 128;       // tokens per CTA (the pair covers 256)
constexpr int BN = 256;       // features per pair tile (MMA N, TMEM columns per accumulator)
constexpr int BNH = BN / 2;   // features whose weights this CTA loads and expands
constexpr int BK = 128;       // int8 elements (= bytes) of K per stage
constexpr int kStages = 6;
constexpr int kAccBufs = 2;
constexpr int kTmemCols = 512;

constexpr int kProducerWarp = 0;
constexpr int kMmaWarp = 1;
// warps 2..5 are the epilogue (one per TMEM lane quarter)
constexpr int kFirstExpanderWarp = 6;
constexpr int kExpanderWarps = (BNH / kTileRows) * (BK / kTileCols); // one warp per packed tile of the stage: 4
constexpr int kThreads = (kFirstExpanderWarp + kExpanderWarps) * 32; // 320

constexpr uint32_t kABytes = BM * BK;   // 16 KiB int8 activations
constexpr uint32_t kBBytes = BNH * BK;  // 16 KiB expanded weights (this CTA's half)
constexpr uint32_t kPBytes = kExpanderWarps * kTileBytes; // 4 KiB packed weights
constexpr uint32_t kStageBytes = kABytes + kBBytes + kPBytes;
constexpr uint32_t kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 512 /*barriers*/;
static_assert(kSmemBytes <= 232448, "exceeds the 227 KiB shared memory of an SM");

struct Barriers {
    uint64_t full[kStages];       // this CTA's TMA bytes landed (activations + packed weights)
    uint64_t expanded[kStages];   // this CTA's weight half written as bytes
    uint64_t ready_peer[kStages]; // leader only: the peer's stage is ready
    uint64_t empty[kStages];      // MMAs that read the stage have completed
    uint64_t acc_full[kAccBufs];  // accumulator complete
    uint64_t acc_empty[kAccBufs]; // leader only: accumulator drained by the epilogues of both CTAs
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
    int tiles_m, tiles_n; // tiles of 256 tokens x 256 features
    int out_i32;
    int32_t *status;
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
prefill_pair_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                    const Params p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u; // swizzled tiles need 1024-byte alignment
    uint8_t *smem = smem_raw + (base - raw);
    // layout: [stage][A | B | P], then the barrier block; identical in both CTAs of the pair
    Barriers *bars = reinterpret_cast<Barriers *>(smem + kStages * kStageBytes);
    volatile int *abort_flag = &bars->abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank(); // 0: leader
    const bool leader = rank == 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&bars->full[s]), 1);
            mbar_init(smem_u32(&bars->expanded[s]), kExpanderWarps);
            mbar_init(smem_u32(&bars->ready_peer[s]), 1);
            mbar_init(smem_u32(&bars->empty[s]), 1);
        }
        for (int b = 0; b < kAccBufs; ++b) {
            mbar_init(smem_u32(&bars->acc_full[b]), 1);
            mbar_init(smem_u32(&bars->acc_empty[b]), 8); // four epilogue warps in each CTA
        }
        bars->abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == kMmaWarp) {
        tmem_alloc_pair(smem_u32(&bars->tmem_base), kTmemCols);
        tmem_relinquish_pair();
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync(); // the peer's barriers are initialised before anything arrives on them
    tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;

    const int n_tiles = p.tiles_m * p.tiles_n;
    const int n_pairs = gridDim.x >> 1, pair = blockIdx.x >> 1;
    const int KB = p.KB;

    if (warp == kProducerWarp) {
        if (lane == 0) {
            prefetch_tensormap(&tmap_x);
            prefetch_tensormap(&tmap_w);
            uint32_t it = 0;
            bool ok = true;
            for (int tile = pair; tile < n_tiles && ok; tile += n_pairs) {
                const int m0 = (tile % p.tiles_m) * (2 * BM) + (int)rank * BM; // this CTA's tokens
                const int n0 = (tile / p.tiles_m) * BN + (int)rank * BNH;      // this CTA's half of the weights
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = it % kStages;
                    const uint32_t round = it / kStages;
                    if (round > 0 && !mbar_wait_bounded(smem_u32(&bars->empty[s]), (round - 1) & 1, abort_flag)) {
                        ok = false;
                        break;
                    }
                    const uint32_t full = smem_u32(&bars->full[s]);
                    const uint32_t a_dst = base + s * kStageBytes;
                    const uint32_t p_dst = a_dst + kABytes + kBBytes;
                    mbar_arrive_expect_tx(full, kABytes + kPBytes);
                    tma_load_2d(a_dst, &tmap_x, kb * BK, m0, full);
                    tma_load_3d(p_dst, &tmap_w, 0, kb * (BK / kTileCols), n0 / kTileRows, full);
                }
            }
        }
    } else if (warp == kMmaWarp) {
        uint32_t it = 0, tile_it = 0;
        bool ok = true;
        if (leader) {
            constexpr uint32_t idesc = idesc_i8(2 * BM, BN, /*a_signed=*/1, /*b_signed=*/0);
            for (int tile = pair; tile < n_tiles && ok; tile += n_pairs, ++tile_it) {
                const int buf = tile_it % kAccBufs;
                const uint32_t use = tile_it / kAccBufs;
                if (use > 0 && !mbar_wait_bounded_cluster(smem_u32(&bars->acc_empty[buf]), (use - 1) & 1, abort_flag)) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = it % kStages;
                    const uint32_t parity = (it / kStages) & 1;
                    if (!mbar_wait_bounded(smem_u32(&bars->full[s]), parity, abort_flag) ||
                        !mbar_wait_bounded(smem_u32(&bars->expanded[s]), parity, abort_flag) ||
                        !mbar_wait_bounded_cluster(smem_u32(&bars->ready_peer[s]), parity, abort_flag)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    if (lane == 0) {
                        const uint32_t a_addr = base + s * kStageBytes;
                        const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
                        for (int k4 = 0; k4 < BK / 32; ++k4) {
                            mma_i8_ss_pair(d_tmem, smem_desc_k_sw128(a_addr + 32 * k4), smem_desc_k_sw128(b_addr + 32 * k4),
                                           idesc, (kb > 0 || k4 > 0) ? 1u : 0u);
                        }
                        mma_commit_pair(smem_u32(&bars->empty[s]), 3); // stage reusable in both CTAs once these MMAs are done
                    }
                    __syncwarp();
                }
                if (ok && lane == 0) mma_commit_pair(smem_u32(&bars->acc_full[buf]), 3);
                __syncwarp();
            }
        } else {
            // relay: when this CTA's half of a stage is complete, tell the leader
            for (int tile = pair; tile < n_tiles && ok; tile += n_pairs) {
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = it % kStages;
                    const uint32_t parity = (it / kStages) & 1;
                    if (!mbar_wait_bounded(smem_u32(&bars->full[s]), parity, abort_flag) ||
                        !mbar_wait_bounded(smem_u32(&bars->expanded[s]), parity, abort_flag)) {
                        ok = false;
                        break;
                    }
                    if (lane == 0) mbar_arrive_remote(map_to_cta(smem_u32(&bars->ready_peer[s]), 0));
                    __syncwarp();
                }
            }
        }
    } else if (warp >= kFirstExpanderWarp) {
        // Expander warp ew owns packed tile (row block ew / 2, column tile ew % 2) of this CTA's half of the
        // stage; layout of a packed tile and the conflict-free choice of slots as in prefill_gemm.cu.
        const int ew = warp - kFirstExpanderWarp;
        const int q = lane >> 3;
        const int g = (lane & 4) ? ((q ^ 1) + 4) : q, tq = lane & 3;
        const int slot = 4 * g + tq;
        const int rbi = ew >> 1, kti = ew & 1;
        uint32_t it = 0;
        bool ok = true;
        for (int tile = pair; tile < n_tiles && ok; tile += n_pairs) {
            for (int kb = 0; kb < KB; ++kb, ++it) {
                const int s = it % kStages;
                const uint32_t parity = (it / kStages) & 1;
                if (!mbar_wait_bounded(smem_u32(&bars->full[s]), parity, abort_flag)) {
                    ok = false;
                    break;
                }
                uint8_t *stage = smem + s * kStageBytes;
                const uint4 *packed = reinterpret_cast<const uint4 *>(stage + kABytes + kBBytes) + ew * (kTileBytes / 16);
                uint8_t *bt = stage + kABytes;
                const uint4 w0 = packed[slot], w1 = packed[32 + slot];
                const uint32_t lo[2][2] = {{w0.x, w0.z}, {w0.y, w0.w}}; // [h][hi], slab 0
                const uint32_t up[2][2] = {{w1.x, w1.z}, {w1.y, w1.w}}; // slab 1
                const int chunk = (kti * 4 + tq) ^ g; // 16-byte chunk of the 128-byte row, swizzled by row % 8 = g
#pragma unroll
                for (int f = 0; f < 4; ++f) {
                    const uint32_t mask = 0x03030303u << (2 * f);
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int r = rbi * kTileRows + 16 * f + 8 * h + g;
                        *reinterpret_cast<uint4 *>(bt + r * 128 + (chunk << 4)) =
                            make_uint4(lo[h][0] & mask, lo[h][1] & mask, up[h][0] & mask, up[h][1] & mask);
                    }
                }
                fence_proxy_async_smem(); // generic-proxy writes -> visible to the tensor cores
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars->expanded[s]));
            }
        }
    } else {
        // epilogue: warp w may touch TMEM lanes 32*(w % 4) .. +31 of this CTA's tensor memory
        const int q = warp & 3;
        uint32_t tile_it = 0;
        const float gamma = p.out_i32 ? 0.0f : *p.gamma;
        const uint32_t acc_empty_leader = map_to_cta(smem_u32(&bars->acc_empty[0]), 0);
        for (int tile = pair; tile < n_tiles; tile += n_pairs, ++tile_it) {
            const int m0 = (tile % p.tiles_m) * (2 * BM) + (int)rank * BM;
            const int n0 = (tile / p.tiles_m) * BN;
            const int buf = tile_it % kAccBufs;
            const uint32_t parity = (tile_it / kAccBufs) & 1;
            if (!mbar_wait_bounded(smem_u32(&bars->acc_full[buf]), parity, abort_flag)) break;
            tc_fence_after_sync();
            const int t = m0 + 32 * q + lane;
            const bool row_ok = t < p.M;
            float scale = 0.0f;
            int rowsum = 0;
            if (row_ok) {
                rowsum = p.rowsum[t];
                if (!p.out_i32) scale = __fdiv_rn(__fmul_rn(gamma, p.beta[t]), (float)kQb);
            }
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t v[32];
                tmem_ld_32x32(tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(buf * BN + c * 32), v);
                tmem_ld_wait();
                const int n = n0 + c * 32;
                // output row n + i carries the factor 4^f, f = ((n + i) % 64) / 16 = 2 (c % 2) + i / 16
                const int sh_lo = 4 * (c & 1), sh_hi = sh_lo + 2;
                int a[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) a[i] = ((int)v[i] >> (i < 16 ? sh_lo : sh_hi)) - rowsum;
                if (row_ok) {
                    if (p.out_i32) {
                        int32_t *dst = reinterpret_cast<int32_t *>(p.out) + (size_t)t * p.N + n;
#pragma unroll
                        for (int i = 0; i < 32; i += 4)
                            if (n + i < p.N) *reinterpret_cast<int4 *>(dst + i) = make_int4(a[i], a[i + 1], a[i + 2], a[i + 3]);
                    } else {
                        __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(p.out) + (size_t)t * p.N + n;
#pragma unroll
                        for (int i = 0; i < 32; i += 8) {
                            if (n + i < p.N) {
                                uint32_t o[4];
#pragma unroll
                                for (int h = 0; h < 4; ++h) {
                                    const float x0 = __fmul_rn((float)a[i + 2 * h], scale);
                                    const float x1 = __fmul_rn((float)a[i + 2 * h + 1], scale);
                                    const __nv_bfloat162 pr = __floats2bfloat162_rn(x0, x1);
                                    o[h] = *reinterpret_cast<const uint32_t *>(&pr);
                                }
                                *reinterpret_cast<uint4 *>(dst + i) = make_uint4(o[0], o[1], o[2], o[3]);
                            }
                        }
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(acc_empty_leader + 8 * buf);
        }
    }

    // common tail: every thread of both CTAs arrives here, also after an expired wait
    if (*abort_flag) {
        if (threadIdx.x == 0) atomicExch(p.status, (int32_t)BITLINEAR_ERR_TIMEOUT);
        // give copies and MMAs that may still be in flight time to land before shared memory and TMEM go away
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync(); // neither CTA leaves while the other may still signal it or use its tensor memory
    if (warp == kMmaWarp) {
        tc_fence_after_sync();
        tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}

// ---- host side ---------------------------------------------------------------------------------

} // namespace

// Number of CTA pairs that can be resident at once (0: the kernel cannot run here).
int prefill_pair_capacity()
{
    static int cached[64] = {0}; // 0 unknown, -1 none
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (cached[dev] == 0) {
        int n = 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2 * (unsigned)sm_count());
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = kSmemBytes;
        if (cudaFuncSetAttribute(prefill_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes) != cudaSuccess ||
            cudaOccupancyMaxActiveClusters(&n, prefill_pair_kernel, &cfg) != cudaSuccess || n <= 0) {
            (void)cudaGetLastError();
            n = -1;
        }
        cached[dev] = n;
    }
    return cached[dev] > 0 ? cached[dev] : 0;
}

cudaError_t launch_prefill_pair(const void *packed, const float *gamma, const int8_t *Xq, const float *beta,
                                const int32_t *rowsum, int64_t M, int64_t K, int64_t N, void *out, int out_i32,
                                WorkspaceHeader *hdr, cudaStream_t stream)
{
    const int capacity = prefill_pair_capacity();
    if (!encode_tiled_fn() || capacity <= 0) return cudaErrorNotSupported;
    const int KB = (int)((K + BK - 1) / BK);

    // activations: box of 128 rows; weights: box of 2 row blocks x 2 column tiles (each CTA expands half a tile)
    CUtensorMap tmap_x, tmap_w;
    if (!encode_activation_map(&tmap_x, Xq, M, K, BM) || !encode_packed_weight_map(&tmap_w, packed, N, K, BNH / kTileRows))
        return cudaErrorInvalidValue;

    Params p;
    p.gamma = gamma;
    p.beta = beta;
    p.rowsum = rowsum;
    p.out = out;
    p.M = (int)M;
    p.N = (int)N;
    p.KB = KB;
    p.tiles_m = (int)((M + 2 * BM - 1) / (2 * BM));
    p.tiles_n = (int)((N + BN - 1) / BN);
    p.out_i32 = out_i32;
    p.status = &hdr->status;

    // One pair per two SMs; pairs beyond what is resident at once (capacity) simply start later: no CTA waits
    // for a CTA outside its own pair.
    int pairs = p.tiles_m * p.tiles_n;
    const int max_pairs = sm_count() / 2;
    if (pairs > max_pairs) pairs = max_pairs;
    prefill_pair_kernel<<<2 * pairs, kThreads, kSmemBytes, stream>>>(tmap_x, tmap_w, p);
    return cudaGetLastError();
}

} // namespace bitlinear
