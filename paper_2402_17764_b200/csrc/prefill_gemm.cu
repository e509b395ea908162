// Kernel (d): ternary x int8 GEMM for many tokens (prefill) on the tcgen05 tensor cores.
//
// With hundreds of tokens every weight is reused hundreds of times, so the integer matmul
// (Section 1 / Section 3 "Energy": matrix multiplication dominates) is a dense contraction and
// belongs on the tensor cores.  Per CTA tile of 128 tokens x 256 output features, per 128-wide
// k block:
//   producer warp  : TMA loads the int8 activation tile (128 x 128 B, 128-byte swizzle) and the
//                    packed 2-bit weight tile (16 row blocks x 512 B) into shared memory;
//   expander warps : turn the 2-bit codes into signed int8 (-1/0/+1) and write them K-major with the
//                    same 128-byte swizzle the tensor core expects;
//   MMA warp       : one thread issues four tcgen05.mma kind::i8 (128 x 256 x 32) per k block into a
//                    TMEM accumulator; tcgen05.commit releases the stage;
//   epilogue warps : tcgen05.ld the finished int32 accumulators, scale by gamma * beta_t / 127,
//                    round to bf16 and store, while the MMA warp fills the second TMEM buffer.
// All waits are bounded; on expiry the CTA sets the workspace status to BITLINEAR_ERR_TIMEOUT,
// every role leaves its loop, TMEM is released and the kernel returns.
//
// Roofline: int8 tensor throughput; algorithmic work 2*M*N*K integer operations.
#include <cuda.h>

#include "internal.cuh"
#include "ptx.cuh"

namespace bitlinear {

namespace {

using namespace ptx;

constexpr int BM = 128;      // tokens per tile  (MMA M, TMEM lanes)
constexpr int BN = 256;      // features per tile (MMA N, TMEM columns per accumulator)
constexpr int BK = 128;      // int8 elements (= bytes) of K per stage
constexpr int kStages = 4;
constexpr int kAccBufs = 2;
constexpr int kTmemCols = 512;

constexpr int kProducerWarp = 0;
constexpr int kMmaWarp = 1;
// warps 2..5 are the epilogue (one per TMEM lane quarter)
constexpr int kFirstExpanderWarp = 6; // 8 warps
constexpr int kExpanderWarps = 8;
constexpr int kThreads = (kFirstExpanderWarp + kExpanderWarps) * 32; // 448

constexpr uint32_t kABytes = BM * BK;            // 16 KiB int8 activations
constexpr uint32_t kBBytes = BN * BK;            // 32 KiB expanded weights
constexpr uint32_t kPBytes = (BN / 16) * 512;    //  8 KiB packed weights
constexpr uint32_t kStageBytes = kABytes + kBBytes + kPBytes;
constexpr uint32_t kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
static_assert(kSmemBytes <= 232448, "exceeds the 227 KiB shared memory of an SM");

struct Barriers {
    uint64_t full[kStages];      // TMA bytes landed (activations + packed weights)
    uint64_t expanded[kStages];  // int8 weight tile written
    uint64_t empty[kStages];     // MMAs that read the stage have completed
    uint64_t acc_full[kAccBufs]; // accumulator complete
    uint64_t acc_empty[kAccBufs];// accumulator drained by the epilogue
    uint32_t tmem_base;
    int abort_flag;
};

struct Params {
    const float *gamma;
    const float *beta;
    void *out;
    int M, N, KB; // KB = padded K / 128
    int tiles_m, tiles_n;
    int out_i32;
    int32_t *status;
};

__device__ __forceinline__ uint32_t expand_signed(uint32_t w, int field)
{
    // 2-bit codes c = T + 1 in each byte's field -> bytes holding T as signed int8:
    // (c + 0x7F) ^ 0x80 maps 0, 1, 2 to 0xFF, 0x00, 0x01 and never carries between bytes.
    return ((((w >> (2 * field)) & 0x03030303u) + 0x7F7F7F7Fu) ^ 0x80808080u);
}

__global__ void __launch_bounds__(kThreads, 1)
prefill_gemm_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                    const Params p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u; // swizzled tiles need 1024-byte alignment
    uint8_t *smem = smem_raw + (base - raw);
    // layout: [stage][A | B | P], then the barrier block
    Barriers *bars = reinterpret_cast<Barriers *>(smem + kStages * kStageBytes);
    volatile int *abort_flag = &bars->abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&bars->full[s]), 1);
            mbar_init(smem_u32(&bars->expanded[s]), kExpanderWarps);
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

    const int n_tiles = p.tiles_m * p.tiles_n;
    const int KB = p.KB;

    if (warp == kProducerWarp) {
        if (lane == 0) {
            prefetch_tensormap(&tmap_x);
            prefetch_tensormap(&tmap_w);
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
                const int m0 = (tile % p.tiles_m) * BM;
                const int n0 = (tile / p.tiles_m) * BN;
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
                    tma_load_2d(a_dst, &tmap_x, kb * BK, m0, full);       // x = byte column (multiple of 128)
                    tma_load_2d(p_dst, &tmap_w, kb * 128, n0 / 16, full); // x = 32-bit word column (multiple of 128)
                }
            }
        }
    } else if (warp == kMmaWarp) {
        constexpr uint32_t idesc = idesc_i8(BM, BN, /*a_signed=*/1, /*b_signed=*/1);
        uint32_t it = 0, tile_it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++tile_it) {
            const int buf = tile_it % kAccBufs;
            const uint32_t use = tile_it / kAccBufs;
            if (use > 0 && !mbar_wait_bounded(smem_u32(&bars->acc_empty[buf]), (use - 1) & 1, abort_flag)) break;
            tc_fence_after_sync();
            const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
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
                    const uint32_t a_addr = base + s * kStageBytes;
                    const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
                    for (int k4 = 0; k4 < BK / 32; ++k4) {
                        mma_i8_ss(d_tmem, smem_desc_k_sw128(a_addr + 32 * k4), smem_desc_k_sw128(b_addr + 32 * k4),
                                  idesc, (kb > 0 || k4 > 0) ? 1u : 0u);
                    }
                    mma_commit(smem_u32(&bars->empty[s])); // stage reusable once these MMAs have read it
                }
                __syncwarp();
            }
            if (ok && lane == 0) mma_commit(smem_u32(&bars->acc_full[buf]));
            __syncwarp();
        }
    } else if (warp >= kFirstExpanderWarp) {
        const int ew = warp - kFirstExpanderWarp;
        const int g = lane >> 2, tq = lane & 3;
        uint32_t it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
            for (int kb = 0; kb < KB; ++kb, ++it) {
                const int s = it % kStages;
                const uint32_t parity = (it / kStages) & 1;
                if (!mbar_wait_bounded(smem_u32(&bars->full[s]), parity, abort_flag)) {
                    ok = false;
                    break;
                }
                uint8_t *stage = smem + s * kStageBytes;
                const uint4 *packed = reinterpret_cast<const uint4 *>(stage + kABytes + kBBytes);
                uint8_t *bt = stage + kABytes;
#pragma unroll
                for (int j = 0; j < (BN / 16) / kExpanderWarps; ++j) {
                    const int rb = ew * ((BN / 16) / kExpanderWarps) + j; // 16-row block inside the tile
                    const uint4 w = packed[rb * 32 + lane];
                    const uint32_t words[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                    for (int half = 0; half < 2; ++half) { // row g, then row g + 8
                        const int r = rb * 16 + g + 8 * half;
                        // 32 columns of this row = two 16-byte chunks, chunk index 2*tq and 2*tq + 1
                        uint4 lo, hi;
                        lo.x = expand_signed(words[0], half);
                        lo.y = expand_signed(words[0], 2 + half);
                        lo.z = expand_signed(words[1], half);
                        lo.w = expand_signed(words[1], 2 + half);
                        hi.x = expand_signed(words[2], half);
                        hi.y = expand_signed(words[2], 2 + half);
                        hi.z = expand_signed(words[3], half);
                        hi.w = expand_signed(words[3], 2 + half);
                        uint8_t *rowp = bt + r * 128;
                        *reinterpret_cast<uint4 *>(rowp + (((2 * tq) ^ (r & 7)) << 4)) = lo;
                        *reinterpret_cast<uint4 *>(rowp + (((2 * tq + 1) ^ (r & 7)) << 4)) = hi;
                    }
                }
                fence_proxy_async_smem(); // generic-proxy writes -> visible to the tensor core
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars->expanded[s]));
            }
        }
    } else {
        // epilogue: warp w may touch TMEM lanes 32*(w % 4) .. +31
        const int q = warp & 3;
        uint32_t tile_it = 0;
        const float gamma = p.out_i32 ? 0.0f : *p.gamma;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++tile_it) {
            const int m0 = (tile % p.tiles_m) * BM;
            const int n0 = (tile / p.tiles_m) * BN;
            const int buf = tile_it % kAccBufs;
            const uint32_t parity = (tile_it / kAccBufs) & 1;
            if (!mbar_wait_bounded(smem_u32(&bars->acc_full[buf]), parity, abort_flag)) break;
            tc_fence_after_sync();
            const int t = m0 + 32 * q + lane;
            const bool row_ok = t < p.M;
            float scale = 0.0f;
            if (row_ok && !p.out_i32) scale = __fdiv_rn(__fmul_rn(gamma, p.beta[t]), (float)kQb);
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t v[32];
                tmem_ld_32x32(tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(buf * BN + c * 32), v);
                tmem_ld_wait();
                const int n = n0 + c * 32;
                if (row_ok) {
                    if (p.out_i32) {
                        int32_t *dst = reinterpret_cast<int32_t *>(p.out) + (size_t)t * p.N + n;
#pragma unroll
                        for (int i = 0; i < 32; i += 4)
                            if (n + i < p.N) *reinterpret_cast<uint4 *>(dst + i) = make_uint4(v[i], v[i + 1], v[i + 2], v[i + 3]);
                    } else {
                        __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(p.out) + (size_t)t * p.N + n;
#pragma unroll
                        for (int i = 0; i < 32; i += 8) {
                            if (n + i < p.N) {
                                uint32_t o[4];
#pragma unroll
                                for (int h = 0; h < 4; ++h) {
                                    const float a = __fmul_rn((float)(int)v[i + 2 * h], scale);
                                    const float b = __fmul_rn((float)(int)v[i + 2 * h + 1], scale);
                                    const __nv_bfloat162 pr = __floats2bfloat162_rn(a, b);
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

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

} // namespace

cudaError_t launch_prefill(const void *packed, const float *gamma, const int8_t *Xq, const float *beta,
                           const int32_t *rowsum, int64_t M, int64_t K, int64_t N, void *out, int out_i32,
                           WorkspaceHeader *hdr, cudaStream_t stream)
{
    (void)rowsum; // signed weight bytes: no offset to remove
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return cudaErrorNotSupported;
    const int KB = (int)((K + kTileCols - 1) / kTileCols);

    CUtensorMap tmap_x, tmap_w;
    {
        // int8 activations [M rows][K bytes]; box 128 bytes x 128 rows; rows/columns past the end read 0
        const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
        const cuuint64_t strides[1] = {(cuuint64_t)K};
        const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)BM};
        const cuuint32_t estr[2] = {1, 1};
        if (encode(&tmap_x, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t *>(Xq), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    {
        // packed weights as [N/16 row blocks][KB * 128 words]; box 128 words (one 512-byte tile) x 16 row blocks
        const cuuint64_t dims[2] = {(cuuint64_t)KB * 128, (cuuint64_t)(N / 16)};
        const cuuint64_t strides[1] = {(cuuint64_t)KB * 512};
        const cuuint32_t box[2] = {128, (cuuint32_t)(BN / 16)};
        const cuuint32_t estr[2] = {1, 1};
        if (encode(&tmap_w, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void *>(packed), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }

    Params p;
    p.gamma = gamma;
    p.beta = beta;
    p.out = out;
    p.M = (int)M;
    p.N = (int)N;
    p.KB = KB;
    p.tiles_m = (int)((M + BM - 1) / BM);
    p.tiles_n = (int)((N + BN - 1) / BN);
    p.out_i32 = out_i32;
    p.status = &hdr->status;

    static bool attr_set[64] = {false};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(prefill_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    int grid = p.tiles_m * p.tiles_n;
    if (grid > sm_count()) grid = sm_count();
    prefill_gemm_kernel<<<grid, kThreads, kSmemBytes, stream>>>(tmap_x, tmap_w, p);
    return cudaGetLastError();
}

} // namespace bitlinear
