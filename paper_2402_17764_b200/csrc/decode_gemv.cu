// Kernel (c): weight-streaming ternary x int8 matmul for M <= 64 tokens (decode).
//
// The cost of decode is moving the weights from HBM once (Section 1: loading weights from DRAM is
// the expensive part; Section 3: time per output token).  All matrices of a launch form ONE sequence
// of 1 KiB tiles (64 output rows x 64 columns each, row block after row block, matrix after matrix),
// and every warp of the grid takes an equal, contiguous share of that sequence.  A warp streams its
// share through a private shared-memory ring filled by bulk copies (cp.async.bulk), so the HBM latency
// is covered by the copy engine and not by registers, and the stream never drains at a row-block or
// matrix boundary.  Row blocks that lie completely inside a share are finished by that warp alone; the
// row blocks cut by the two ends of a share are completed through int32 atomics (exact, order-free) by
// whichever contributor arrives last.
//
// The inner loop is bound by integer-ALU issue, not by the tensor pipe, so the 2-bit codes are never
// shifted into place.  One byte of the packed format holds the codes of FOUR ROWS at the same column
// (field f = bits 2f, 2f+1 belongs to row 16 f + r), and the four 32-bit words a lane loads with one
// 16-byte shared-memory load are, as they are, the A operand of the warp-level integer MMA
// (u8 x s8 -> s32).  Four MMAs take these operands:
//     w                 bytes  c0 + 4 c1 + 16 c2 + 64 c3      (the loaded registers, no instruction)
//     w & 0xFCFCFCFC    bytes       4 c1 + 16 c2 + 64 c3
//     w & 0xF0F0F0F0    bytes              16 c2 + 64 c3
//     w & 0xC0C0C0C0    bytes                      64 c3
// Every byte is a valid u8 (<= 170).  The four accumulators then hold the linear combinations
//     a0 = S0 + 4 S1 + 16 S2 + 64 S3,  a1 = 4 (S1 + 4 S2 + 16 S3),  a2 = 16 (S2 + 4 S3),  a3 = 64 S3
// of the four row sums S_f = sum_k code_f(k) q(k), which are separated again, exactly, once per row
// block.  Because codes are T + 1, the per-token sum of q is subtracted once at the end.
//
// Roofline: HBM.  Algorithmic bytes = N*K/4 per matrix (activations and outputs are < 0.1 % at M = 1).
#include "internal.cuh"
#include "ptx.cuh"

namespace bitlinear {

namespace {

// Tuning constants (the defaults were chosen by measurement on B200; the macros exist for sweeps).
#ifndef BITLINEAR_DECODE_WARPS
#define BITLINEAR_DECODE_WARPS 8
#endif
#ifndef BITLINEAR_DECODE_CHUNK_TILES
#define BITLINEAR_DECODE_CHUNK_TILES 8
#endif
#ifndef BITLINEAR_DECODE_STAGES
#define BITLINEAR_DECODE_STAGES 2
#endif
#ifndef BITLINEAR_DECODE_CTAS_PER_SM
#define BITLINEAR_DECODE_CTAS_PER_SM 1
#endif
constexpr int kWarps = BITLINEAR_DECODE_WARPS;             // warps per CTA, each independent
constexpr int kChunkTiles = BITLINEAR_DECODE_CHUNK_TILES;  // tiles per bulk copy
constexpr int kChunkBytes = kChunkTiles * kTileBytes;
constexpr int kStages = BITLINEAR_DECODE_STAGES;           // copies in flight per warp
constexpr int kRingBytes = kWarps * kStages * kChunkBytes; // per CTA
constexpr int kDecodeSmem = kRingBytes + kWarps * kStages * 8 + 16;
constexpr int kCtasPerSm = BITLINEAR_DECODE_CTAS_PER_SM;

__device__ __forceinline__ void mma_u8s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// unsigned bytes (codes) x signed bytes (activations), accumulated in int32
__device__ __forceinline__ int dp4a_u8s8(uint32_t a, uint32_t b, int c)
{
    int d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

__device__ __forceinline__ uint4 ld_stream(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// Entry that owns tile t of the launch-wide sequence: the last one whose tile_begin <= t.
// All lanes of the warp search together, so the lookup costs one round of loads.
__device__ __forceinline__ int find_entry(const DecodeEntry *tab, int n_entries, uint32_t t, int lane)
{
    int best = 0;
    for (int i = lane; i < n_entries; i += 32)
        if (tab[i].tile_begin <= t) best = i; // entries are in ascending order
    return __reduce_max_sync(0xffffffffu, best);
}

// Writes one finished row sum: raw int32 (test hook) or dequantised bf16.
__device__ __forceinline__ void store_result(const DecodeEntry &e, int token, int row, int dot_codes, int rowsum,
                                             float scale)
{
    const int acc = dot_codes - rowsum; // sum_k (T+1) q - sum_k q
    const size_t idx = (size_t)token * e.N + row;
    if (e.out_i32) {
        reinterpret_cast<int32_t *>(e.out)[idx] = acc;
    } else {
        reinterpret_cast<__nv_bfloat16 *>(e.out)[idx] = __float2bfloat16_rn(__fmul_rn((float)acc, scale));
    }
}

__device__ __forceinline__ float token_scale(const DecodeEntry &e, int token)
{
    if (e.out_i32) return 0.0f;
    return __fdiv_rn(__fmul_rn(*e.gamma, e.beta[token]), (float)kQb); // (gamma * beta_t) / Qb
}

// End of a row block.  `each(fn)` calls fn(token, row, partial row sum) for every output this lane holds;
// `tiles` of the row block's KB column tiles went into the sums.  If that is all of them the sums are
// final.  Otherwise partial sums meet in the int32 scratch and the contributor that brings the tile count
// to KB finishes the row block and leaves scratch and counter clean for the next launch.
template <class Each>
__device__ __forceinline__ void finish_block(const DecodeEntry &e, int rb, int tiles, int lane, Each each)
{
    if (tiles == e.KB) {
        each([&](int token, int row, int v) { store_result(e, token, row, v, e.rowsum[token], token_scale(e, token)); });
        return;
    }
    each([&](int token, int row, int v) { atomicAdd(&e.acc32[(size_t)token * e.N + row], v); });
    __threadfence();
    __syncwarp();
    uint32_t old = 0;
    if (lane == 0) old = atomicAdd(&e.counters[rb], (uint32_t)tiles);
    old = __shfl_sync(0xffffffffu, old, 0);
    if (old + (uint32_t)tiles != (uint32_t)e.KB) return;
    __threadfence();
    each([&](int token, int row, int) {
        int32_t *p = &e.acc32[(size_t)token * e.N + row];
        const int total = __ldcg(p);
        __stcg(p, 0);
        store_result(e, token, row, total, e.rowsum[token], token_scale(e, token));
    });
    if (lane == 0) e.counters[rb] = 0u;
}

// ---------------------------------------------------------------------------------------------
// Integer-MMA path.  NT = number of 8-token column tiles (M <= 8 * NT).
//
// A tile is two slabs of 512 bytes (columns 8 s .. 8 s + 7 of every 16-column group, s = 0, 1).  Lane
// (g = lane / 4, tq = lane % 4) holds 16 bytes of each slab: word j, byte b, field f is
//     row 16 f + 8 (j % 2) + g,   column 16 tq + 8 s + 4 (j / 2) + b      of the tile,
// which is exactly the A fragment of mma.m16n8k32 (a0: row g, k 4tq..; a1: row g + 8; a2, a3: k + 16) for
// the 16 rows of field f.  The B fragment of lane (g, tq) is token g, columns 16 tq .. 16 tq + 15: one
// 16-byte load serves both slabs.

__device__ __forceinline__ void mma_slab(int (&acc)[4][4], const uint4 &w, uint32_t b0, uint32_t b1)
{
    mma_u8s8(acc[0], w.x, w.y, w.z, w.w, b0, b1);
    mma_u8s8(acc[1], w.x & 0xFCFCFCFCu, w.y & 0xFCFCFCFCu, w.z & 0xFCFCFCFCu, w.w & 0xFCFCFCFCu, b0, b1);
    mma_u8s8(acc[2], w.x & 0xF0F0F0F0u, w.y & 0xF0F0F0F0u, w.z & 0xF0F0F0F0u, w.w & 0xF0F0F0F0u, b0, b1);
    mma_u8s8(acc[3], w.x & 0xC0C0C0C0u, w.y & 0xC0C0C0C0u, w.z & 0xC0C0C0C0u, w.w & 0xC0C0C0C0u, b0, b1);
}

__device__ __forceinline__ void mma_tile(int (&acc)[4][4], uint32_t stage, const uint4 &x)
{
    mma_slab(acc, lds128(stage), x.x, x.y);
    mma_slab(acc, lds128(stage + 512), x.z, x.w);
}

__device__ __forceinline__ uint4 load_x16(const int8_t *p) { return __ldg(reinterpret_cast<const uint4 *>(p)); }

template <int NT>
__global__ void __launch_bounds__(kWarps * 32, (NT <= 2) ? kCtasPerSm : 1) decode_mma_kernel(
    const __grid_constant__ InlineTable inl, const DecodeEntry *__restrict__ table, int n_entries,
    uint32_t total_tiles, WorkspaceHeader *hdr)
{
    extern __shared__ __align__(128) uint8_t dsmem[];
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3;
    const uint32_t ring = ptx::smem_u32(dsmem) + warp * (kStages * kChunkBytes);
    const uint32_t ring_lane = ring + lane * 16;
    const uint32_t bars = ptx::smem_u32(dsmem + kRingBytes) + warp * (kStages * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(dsmem + kRingBytes + kWarps * kStages * 8);

    if (threadIdx.x == 0) *abort_flag = 0;
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < kStages; ++s) ptx::mbar_init(bars + 8 * s, 1);
        ptx::fence_mbar_init();
    }
    __syncthreads();

    const DecodeEntry *tab = table ? table : inl.e;
    // this warp's share of the tile sequence
    const uint64_t n_warps = (uint64_t)gridDim.x * kWarps, w = (uint64_t)blockIdx.x * kWarps + warp;
    const uint32_t t_begin = (uint32_t)((uint64_t)total_tiles * w / n_warps);
    const uint32_t t_end = (uint32_t)((uint64_t)total_tiles * (w + 1) / n_warps);
    if (t_begin == t_end) return;

    // Two cursors walk the share: the producer issues copies up to kStages chunks ahead of the consumer.
    // A chunk is up to kChunkTiles tiles and never crosses the end of a row block, so both cursors cut the
    // share into the same chunks.
    const DecodeEntry *pe = tab + find_entry(tab, n_entries, t_begin, lane);
    const DecodeEntry *e = pe;
    int KB = e->KB;
    int rb, kt;
    {
        const uint32_t local = t_begin - e->tile_begin;
        rb = (int)(local / (uint32_t)KB);
        kt = (int)(local - (uint32_t)rb * (uint32_t)KB);
    }
    int left = (int)(t_end - t_begin);                  // consumer: tiles left in the share
    int p_left = left, p_kt = kt, p_KB = KB;            // producer: same, plus its place in the row block
    int p_blocks = e->NB - rb;                          // producer: row blocks left in its matrix, this one included
    const uint8_t *p_src = reinterpret_cast<const uint8_t *>(e->packed) + ((size_t)rb * KB + kt) * kTileBytes;
    uint32_t issued = 0, consumed = 0;                  // chunks, over the whole kernel (ring slot = count % kStages)

    auto top_up = [&]() {
        while (p_left > 0 && issued - consumed < (uint32_t)kStages) {
            const int n = min(min(kChunkTiles, p_KB - p_kt), p_left);
            if (lane == 0) {
                const uint32_t s = issued % kStages;
                ptx::mbar_arrive_expect_tx(bars + 8 * s, (uint32_t)n * kTileBytes);
                bulk_copy_g2s(ring + s * kChunkBytes, p_src, (uint32_t)n * kTileBytes, bars + 8 * s);
            }
            ++issued;
            p_left -= n;
            p_kt += n;
            p_src += (size_t)n * kTileBytes;
            if (p_kt == p_KB) {
                p_kt = 0;
                if (--p_blocks == 0 && p_left > 0) { // next matrix
                    ++pe;
                    p_KB = pe->KB;
                    p_blocks = pe->NB;
                    p_src = reinterpret_cast<const uint8_t *>(pe->packed);
                }
            }
        }
    };
    top_up();

    bool alive = true;
    while (alive && left > 0) {
        // ---- one row block (or the part of it that lies in this share)
        const int K = e->K, M = e->M;
        int acc[NT][4][4];      // [token tile][field][C fragment]
        const int8_t *xrow[NT]; // this lane's B-fragment token: lanes whose token does not exist read the last one
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
            for (int f = 0; f < 4; ++f) acc[nt][f][0] = acc[nt][f][1] = acc[nt][f][2] = acc[nt][f][3] = 0;
            xrow[nt] = e->Xq + (size_t)min(8 * nt + g, M - 1) * K + 16 * tq;
        }
        int tiles = 0; // tiles of this row block accumulated here
        while (kt < KB && left > 0) {
            const int n = min(min(kChunkTiles, KB - kt), left);
            const uint32_t s = consumed % kStages;
            const uint32_t stage = ring_lane + s * kChunkBytes;
            const int col0 = kt * kTileCols + 16 * tq; // this lane's first column; columns >= K read as zero
            if (NT == 1) {
                // activations of the whole chunk are requested before the weights are waited for
                uint4 x[kChunkTiles];
                const int8_t *xp = xrow[0] + kt * kTileCols;
                // (the condition must be the same for all lanes: mma.sync needs the whole warp)
                if (n == kChunkTiles && (kt + kChunkTiles) * kTileCols <= K) {
#pragma unroll
                    for (int t = 0; t < kChunkTiles; ++t) x[t] = load_x16(xp + t * kTileCols);
                    if (!ptx::mbar_wait_bounded(bars + 8 * s, (consumed / kStages) & 1u, abort_flag)) { alive = false; break; }
#pragma unroll
                    for (int t = 0; t < kChunkTiles; ++t) mma_tile(acc[0], stage + t * kTileBytes, x[t]);
                } else {
#pragma unroll
                    for (int t = 0; t < kChunkTiles; ++t) {
                        x[t] = make_uint4(0u, 0u, 0u, 0u);
                        if (t < n && col0 + t * kTileCols < K) x[t] = load_x16(xp + t * kTileCols);
                    }
                    if (!ptx::mbar_wait_bounded(bars + 8 * s, (consumed / kStages) & 1u, abort_flag)) { alive = false; break; }
#pragma unroll
                    for (int t = 0; t < kChunkTiles; ++t)
                        if (t < n) mma_tile(acc[0], stage + t * kTileBytes, x[t]);
                }
            } else {
                if (!ptx::mbar_wait_bounded(bars + 8 * s, (consumed / kStages) & 1u, abort_flag)) { alive = false; break; }
#pragma unroll
                for (int t = 0; t < kChunkTiles; ++t) {
                    if (t < n) {
                        const uint4 w0 = lds128(stage + t * kTileBytes);
                        const uint4 w1 = lds128(stage + t * kTileBytes + 512);
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            uint4 x = make_uint4(0u, 0u, 0u, 0u);
                            if (col0 + t * kTileCols < K) x = load_x16(xrow[nt] + kt * kTileCols + t * kTileCols);
                            mma_slab(acc[nt], w0, x.x, x.y);
                            mma_slab(acc[nt], w1, x.z, x.w);
                        }
                    }
                }
            }
            __syncwarp(); // every lane has read the slot before lane 0 refills it
            ++consumed;
            kt += n;
            tiles += n;
            left -= n;
            top_up();
        }
        if (!alive) break;

        // C fragment of field f: c0 (row 16f + g, token 2tq), c1 (same row, 2tq + 1), c2 (row 16f + 8 + g, 2tq), c3.
        const int N = e->N, row0 = rb * kTileRows + g;
        finish_block(*e, rb, tiles, lane, [&](auto fn) {
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
                for (int tb = 0; tb < 2; ++tb) {
                    const int token = 8 * nt + 2 * tq + tb;
                    if (token >= M) continue;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int c = 2 * h + tb;
                        const int t1 = acc[nt][1][c] >> 2; // S1 + 4 S2 + 16 S3   (exact shifts)
                        const int t2 = acc[nt][2][c] >> 4; // S2 + 4 S3
                        const int t3 = acc[nt][3][c] >> 6; // S3
                        const int S[4] = {acc[nt][0][c] - 4 * t1, t1 - 4 * t2, t2 - 4 * t3, t3};
#pragma unroll
                        for (int f = 0; f < 4; ++f) {
                            const int r = row0 + 16 * f + 8 * h;
                            if (r < N) fn(token, r, S[f]);
                        }
                    }
                }
            }
        });

        // next row block, or next matrix
        if (kt == KB) {
            kt = 0;
            if (++rb == e->NB && left > 0) {
                ++e;
                rb = 0;
                KB = e->KB;
            }
        }
    }
    if (*abort_flag) {
        if (lane == 0) atomicExch(&hdr->status, (int32_t)BITLINEAR_ERR_TIMEOUT);
        // let copies that may still be in flight land before the ring goes away
        const uint64_t t0 = ptx::globaltimer_ns();
        while (ptx::globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
}

// ---------------------------------------------------------------------------------------------
// dp4a path (M <= 8, one matrix): one warp per row block over the whole K, plain loads, shift-and-mask
// unpacking, scalar dot products; each lane multiplies its own 8 rows x 16 columns, then the four
// lanes that share the rows add up with two shuffles.  Kept as an independent cross-check of the MMA path.
__global__ void __launch_bounds__(kWarps * 32) decode_dp4a_kernel(const __grid_constant__ InlineTable inl)
{
    const DecodeEntry &e = inl.e[0];
    const int lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3;
    const int K = e.K, M = e.M, KB = e.KB;
    for (int rb = blockIdx.x * kWarps + (threadIdx.x >> 5); rb < e.NB; rb += gridDim.x * kWarps) {
        int acc[8][2][4]; // [token][row half][field]
#pragma unroll
        for (int t = 0; t < 8; ++t)
#pragma unroll
            for (int h = 0; h < 2; ++h) acc[t][h][0] = acc[t][h][1] = acc[t][h][2] = acc[t][h][3] = 0;
        const uint4 *wp = e.packed + (size_t)rb * KB * (kTileBytes / 16) + lane;
        for (int kt = 0; kt < KB; ++kt, wp += kTileBytes / 16) {
            const uint4 w0 = ld_stream(wp), w1 = ld_stream(wp + 32);
            // [slab][word]: word j is row half j % 2, columns 8 slab + 4 (j / 2) .. + 3 of this lane's 16
            const uint32_t words[2][4] = {{w0.x, w0.y, w0.z, w0.w}, {w1.x, w1.y, w1.z, w1.w}};
            const int col = kt * kTileCols + 16 * tq;
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                if (t >= M) break;
                uint4 xa = make_uint4(0u, 0u, 0u, 0u);
                if (col < K) xa = __ldg(reinterpret_cast<const uint4 *>(e.Xq + (size_t)t * K + col));
                const uint32_t xs[4] = {xa.x, xa.y, xa.z, xa.w};
#pragma unroll
                for (int sl = 0; sl < 2; ++sl)
#pragma unroll
                    for (int j = 0; j < 4; ++j)
#pragma unroll
                        for (int f = 0; f < 4; ++f)
                            acc[t][j & 1][f] = dp4a_u8s8((words[sl][j] >> (2 * f)) & 0x03030303u, xs[2 * sl + (j >> 1)],
                                                         acc[t][j & 1][f]);
            }
        }
        const int N = e.N, row0 = rb * kTileRows + g;
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            if (t >= M) break;
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int f = 0; f < 4; ++f) {
                    int v = acc[t][h][f];
                    v += __shfl_xor_sync(0xffffffffu, v, 1);
                    v += __shfl_xor_sync(0xffffffffu, v, 2);
                    const int r = row0 + 16 * f + 8 * h;
                    if (tq == 0 && r < N) store_result(e, t, r, v, e.rowsum[t], token_scale(e, t));
                }
        }
    }
}

} // namespace

template <int NT>
static cudaError_t launch_mma(dim3 grid, dim3 block, const InlineTable &inl, const DecodeEntry *table, int n_entries,
                              uint32_t total_tiles, WorkspaceHeader *hdr, cudaStream_t stream)
{
    static bool attr_set[64] = {false};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(decode_mma_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDecodeSmem);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    decode_mma_kernel<NT><<<grid, block, kDecodeSmem, stream>>>(inl, table, n_entries, total_tiles, hdr);
    return cudaGetLastError();
}

cudaError_t launch_decode(const InlineTable &inl, const DecodeEntry *table, int n_entries, uint32_t total_tiles,
                          int max_M, int path, WorkspaceHeader *hdr, cudaStream_t stream)
{
    if (total_tiles == 0) return cudaSuccess;
    const dim3 block(kWarps * 32);
    if (path == BITLINEAR_PATH_DP4A) {
        int ctas = (inl.e[0].NB + kWarps - 1) / kWarps;
        const int cap = sm_count() * 4;
        if (ctas > cap) ctas = cap;
        decode_dp4a_kernel<<<dim3(ctas), block, 0, stream>>>(inl);
        return cudaGetLastError();
    }
    // every warp should have at least kMinTilesPerWarp tiles; beyond that, fill the machine
    constexpr uint32_t kMinTilesPerWarp = 4;
    uint32_t ctas = (total_tiles + kMinTilesPerWarp * kWarps - 1) / (kMinTilesPerWarp * kWarps);
    const uint32_t cap = (uint32_t)sm_count() * (max_M <= 16 ? kCtasPerSm : 1);
    if (ctas > cap) ctas = cap;
    const dim3 grid(ctas);
    if (max_M <= 8) return launch_mma<1>(grid, block, inl, table, n_entries, total_tiles, hdr, stream);
    if (max_M <= 16) return launch_mma<2>(grid, block, inl, table, n_entries, total_tiles, hdr, stream);
    if (max_M <= 32) return launch_mma<4>(grid, block, inl, table, n_entries, total_tiles, hdr, stream);
    return launch_mma<8>(grid, block, inl, table, n_entries, total_tiles, hdr, stream);
}

} // namespace bitlinear
