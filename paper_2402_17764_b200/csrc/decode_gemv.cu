// Kernel (c): weight-streaming ternary x int8 matmul for M <= 64 tokens (decode).
//
// The cost of decode is moving the weights from HBM once (Section 1: loading weights from DRAM is
// the expensive part; Section 3: time per output token).  Each warp owns work units of
// 16 output rows x a range of 128-column tiles.  It streams the 512-byte packed tiles with one
// 16-byte load per lane, turns every 32-bit word into four integer-MMA operand registers with a
// shift and a mask (codes 0/1/2 as unsigned bytes), and multiplies them against int8 activations
// with mma.sync m16n8k32 (u8 x s8 -> s32): the tensor core does the k reduction across lanes, so no
// shuffles are needed.  Because codes are T + 1, the per-token row sum is subtracted once at the end.
// Units are handed out dynamically over ALL matrices of a launch, so a whole decode step (hundreds
// of small matrices) streams without gaps between matrices.
//
// Roofline: HBM.  Algorithmic bytes = N*K/4 per matrix (activations and outputs are < 0.1 % at M = 1).
#include "internal.cuh"
#include "ptx.cuh"

namespace bitlinear {

namespace {

constexpr int kWarps = 8;          // warps per CTA, each independent
constexpr int kTilesInFlight = 4;  // 16-byte loads per lane issued before the first is consumed

__device__ __forceinline__ uint4 ld_stream(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

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

// Dynamic work distribution.  The units are dealt into n_stripes interleaved stripes (stripe c owns
// units c, c + n_stripes, ...), each with its own counter; a warp draws only from its home stripe
// (global warp index mod n_stripes) and stops when that stripe is empty.  Every stripe has at least one
// home warp because n_stripes <= number of warps.  The draw for the NEXT unit is issued before the
// current unit is processed, so the atomic's latency is hidden.
struct UnitQueue {
    uint32_t *counter;
    uint32_t total, n_stripes, stripe;
    uint32_t pending; // result of the draw in flight (lane 0)

    __device__ __forceinline__ void init(WorkspaceHeader *h, uint32_t total_units, uint32_t stripes,
                                         uint32_t global_warp, int lane)
    {
        total = total_units;
        n_stripes = stripes;
        stripe = global_warp % stripes;
        counter = &h->unit_counter[stripe][0];
        draw(lane);
    }
    __device__ __forceinline__ void draw(int lane)
    {
        if (lane == 0) pending = atomicAdd(counter, 1u);
    }
    // Returns the next unit index, or 0xFFFFFFFF when the stripe is empty; leaves a new draw in flight.
    __device__ __forceinline__ uint32_t next(int lane)
    {
        const uint32_t i = __shfl_sync(0xffffffffu, pending, 0);
        const uint64_t unit = (uint64_t)i * n_stripes + stripe;
        if (unit >= total) return 0xFFFFFFFFu;
        draw(lane);
        return (uint32_t)unit;
    }
};

// Writes one finished accumulator: raw int32 (test hook) or dequantised bf16.
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

// Entry that owns a unit: the last one whose unit_begin <= unit.
__device__ __forceinline__ int find_entry(const DecodeEntry *tab, int n_entries, int unit)
{
    int lo = 0, hi = n_entries - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (tab[mid].unit_begin <= unit) lo = mid; else hi = mid - 1;
    }
    return lo;
}

struct UnitCoords {
    int rb, kt0, kt1, split;
};

__device__ __forceinline__ UnitCoords unit_coords(const DecodeEntry &e, uint32_t unit)
{
    UnitCoords u;
    const int local = (int)unit - e.unit_begin;
    u.rb = local / e.ksplit;
    u.split = local - u.rb * e.ksplit;
    u.kt0 = (int)((long long)e.KB * u.split / e.ksplit);
    u.kt1 = (int)((long long)e.KB * (u.split + 1) / e.ksplit);
    return u;
}

// Split-K tail: add partial sums to the scratch, and let the last split to arrive finish the rows.
// vals[i] belongs to (token tok[i], row row[i]); invalid slots have tok[i] < 0.
template <int NV>
__device__ __forceinline__ void finish_unit(const DecodeEntry &e, const UnitCoords &u, int lane, const int (&vals)[NV],
                                            const int (&tok)[NV], const int (&row)[NV])
{
    if (e.ksplit == 1) {
#pragma unroll
        for (int i = 0; i < NV; ++i)
            if (tok[i] >= 0) store_result(e, tok[i], row[i], vals[i], e.rowsum[tok[i]], token_scale(e, tok[i]));
        return;
    }
#pragma unroll
    for (int i = 0; i < NV; ++i)
        if (tok[i] >= 0) atomicAdd(&e.acc32[(size_t)tok[i] * e.N + row[i]], vals[i]);
    __threadfence();
    __syncwarp();
    uint32_t old = 0;
    if (lane == 0) old = atomicAdd(&e.counters[u.rb], 1u);
    old = __shfl_sync(0xffffffffu, old, 0);
    if (old != (uint32_t)e.ksplit - 1u) return;
    __threadfence();
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        if (tok[i] >= 0) {
            int32_t *p = &e.acc32[(size_t)tok[i] * e.N + row[i]];
            const int total = __ldcg(p);
            __stcg(p, 0); // leave the scratch clean for the next launch
            store_result(e, tok[i], row[i], total, e.rowsum[tok[i]], token_scale(e, tok[i]));
        }
    }
    if (lane == 0) e.counters[u.rb] = 0u;
}

// ---------------------------------------------------------------------------------------------
// Integer-MMA path.  NT = number of 8-token column tiles (M <= 8 * NT).
//
// Each warp owns a private ring of kStages x 2 KiB in shared memory.  Lane 0 keeps up to kStages
// bulk copies (cp.async.bulk, 4 tiles = 2 KiB each) in flight; completion is counted on one mbarrier
// per stage.  The HBM latency is therefore hidden by the copy engine, not by registers.
//
// The loop is bound by integer-ALU issue, so unpacking is kept to 5 logic instructions per 16 weights:
// the low two fields of each byte are masked where they sit,
//     t  = w >> 4
//     a0 = w & 0x03030303   a1 = w & 0x0C0C0C0C   a2 = t & 0x03030303   a3 = t & 0x0C0C0C0C
// so the bytes of a1 and a3 (rows g + 8) hold 4 * code (<= 8, a valid u8) and rows g + 8 of the
// accumulator come out multiplied by 4; one exact arithmetic shift per work unit undoes that.
constexpr int kStages = 4;
constexpr int kGroupTiles = 4;
constexpr int kGroupBytes = kGroupTiles * kTileBytes;
constexpr int kRingBytes = kWarps * kStages * kGroupBytes; // 64 KiB per CTA
constexpr int kDecodeSmem = kRingBytes + kWarps * kStages * 8 + 16;

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

// 32 int8 activations (columns col .. col+31 of one token) as eight registers.
struct X32 {
    uint4 a, b;
};

__device__ __forceinline__ X32 load_x32(const int8_t *p)
{
    X32 x;
    x.a = __ldg(reinterpret_cast<const uint4 *>(p));
    x.b = __ldg(reinterpret_cast<const uint4 *>(p + 16));
    return x;
}

// Same, for the last tile of a matrix whose K is not a multiple of 128: columns >= K read as zero
// (the padded weight columns hold code 1, so the activation there must be 0).
__device__ __forceinline__ X32 load_x32_ragged(const int8_t *p, int col, int K)
{
    X32 x;
    x.a = make_uint4(0u, 0u, 0u, 0u);
    x.b = make_uint4(0u, 0u, 0u, 0u);
    if (col < K) x.a = __ldg(reinterpret_cast<const uint4 *>(p));
    if (col + 16 < K) x.b = __ldg(reinterpret_cast<const uint4 *>(p + 16));
    return x;
}

// One 16 x 128 tile (this lane's four words) against one 8-token column tile.
__device__ __forceinline__ void mma_tile(int (&acc0)[4], int (&acc1)[4], const uint4 &w, const X32 &x)
{
    const uint32_t lo = 0x03030303u, hi = 0x0C0C0C0Cu;
    uint32_t t;
    t = w.x >> 4;
    mma_u8s8(acc0, w.x & lo, w.x & hi, t & lo, t & hi, x.a.x, x.a.y);
    t = w.y >> 4;
    mma_u8s8(acc1, w.y & lo, w.y & hi, t & lo, t & hi, x.a.z, x.a.w);
    t = w.z >> 4;
    mma_u8s8(acc0, w.z & lo, w.z & hi, t & lo, t & hi, x.b.x, x.b.y);
    t = w.w >> 4;
    mma_u8s8(acc1, w.w & lo, w.w & hi, t & lo, t & hi, x.b.z, x.b.w);
}

template <int NT>
__global__ void __launch_bounds__(kWarps * 32, (NT <= 2) ? 3 : ((NT == 4) ? 2 : 1)) decode_mma_kernel(
    const __grid_constant__ InlineTable inl, const DecodeEntry *__restrict__ table, int n_entries, int total_units,
    int n_stripes, WorkspaceHeader *hdr)
{
    extern __shared__ __align__(128) uint8_t dsmem[];
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3;
    const uint32_t ring = ptx::smem_u32(dsmem) + warp * (kStages * kGroupBytes);
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
    uint32_t issued = 0, consumed = 0; // 2 KiB groups, counted over the whole kernel (stage = count % kStages)
    UnitQueue queue;
    queue.init(hdr, (uint32_t)total_units, (uint32_t)n_stripes, blockIdx.x * kWarps + warp, lane);
    bool alive = true;
    while (alive) {
        const uint32_t unit = queue.next(lane);
        if (unit == 0xFFFFFFFFu) break;
        const int ei = find_entry(tab, n_entries, (int)unit);
        const DecodeEntry &e = tab[ei];
        const UnitCoords u = unit_coords(e, unit);
        const int K = e.K;
        const int n_tiles = u.kt1 - u.kt0;
        const int n_groups = (n_tiles + kGroupTiles - 1) / kGroupTiles;
        const uint8_t *src = reinterpret_cast<const uint8_t *>(e.packed) + ((size_t)u.rb * e.KB + u.kt0) * kTileBytes;

        auto issue_group = [&](int j) {
            if (lane == 0) {
                const int tiles = min(kGroupTiles, n_tiles - j * kGroupTiles);
                const uint32_t s = issued % kStages;
                ptx::mbar_arrive_expect_tx(bars + 8 * s, (uint32_t)tiles * kTileBytes);
                bulk_copy_g2s(ring + s * kGroupBytes, src + (size_t)j * kGroupBytes, (uint32_t)tiles * kTileBytes,
                              bars + 8 * s);
            }
            ++issued;
        };
        for (int j = 0; j < n_groups && j < kStages; ++j) issue_group(j);

        int acc[NT][2][4]; // [token tile][copy (breaks the MMA dependency chain)][C fragment]
        const int8_t *xp[NT]; // this lane's 32 columns of its B-fragment token, at the unit's first tile
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
            for (int c = 0; c < 2; ++c) acc[nt][c][0] = acc[nt][c][1] = acc[nt][c][2] = acc[nt][c][3] = 0;
            // lanes whose token does not exist read the last token instead; their columns are discarded below
            const int token = min(8 * nt + g, e.M - 1);
            xp[nt] = e.Xq + (size_t)token * K + (size_t)u.kt0 * kTileCols + 32 * tq;
        }
        // tiles that lie completely inside K take the fast path
        const int full_tiles = min(n_tiles, K / kTileCols - u.kt0);

        for (int j = 0; j < n_groups; ++j) {
            const int t0 = j * kGroupTiles;
            const uint32_t s = consumed % kStages;
            const uint32_t stage = ring_lane + s * kGroupBytes;
            if (t0 + kGroupTiles <= full_tiles) {
                if (NT == 1) {
                    // activations of the whole group are requested before the weights are waited for
                    X32 x[kGroupTiles];
#pragma unroll
                    for (int t = 0; t < kGroupTiles; ++t) x[t] = load_x32(xp[0] + (t0 + t) * kTileCols);
                    if (!ptx::mbar_wait_bounded(bars + 8 * s, (consumed / kStages) & 1u, abort_flag)) { alive = false; break; }
#pragma unroll
                    for (int t = 0; t < kGroupTiles; ++t)
                        mma_tile(acc[0][0], acc[0][1], lds128(stage + t * kTileBytes), x[t]);
                } else {
                    if (!ptx::mbar_wait_bounded(bars + 8 * s, (consumed / kStages) & 1u, abort_flag)) { alive = false; break; }
#pragma unroll
                    for (int t = 0; t < kGroupTiles; ++t) {
                        const uint4 w = lds128(stage + t * kTileBytes);
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt)
                            mma_tile(acc[nt][0], acc[nt][1], w, load_x32(xp[nt] + (t0 + t) * kTileCols));
                    }
                }
            } else {
                // last, short or ragged group of the unit
                const int tiles = min(kGroupTiles, n_tiles - t0);
                if (!ptx::mbar_wait_bounded(bars + 8 * s, (consumed / kStages) & 1u, abort_flag)) { alive = false; break; }
                for (int t = 0; t < tiles; ++t) {
                    const uint4 w = lds128(stage + t * kTileBytes);
                    const int col = (u.kt0 + t0 + t) * kTileCols + 32 * tq;
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt)
                        mma_tile(acc[nt][0], acc[nt][1], w, load_x32_ragged(xp[nt] + (t0 + t) * kTileCols, col, K));
                }
            }
            __syncwarp(); // every lane has read the stage before lane 0 refills it
            ++consumed;
            if (j + kStages < n_groups) issue_group(j + kStages);
        }
        if (!alive) break;

        // C fragment: c0 (row g, token 2tq), c1 (row g, token 2tq+1), c2 (row g+8, token 2tq), c3 (row g+8, 2tq+1)
        int vals[NT * 4], tok[NT * 4], row[NT * 4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int sum = acc[nt][0][c] + acc[nt][1][c];
                const int token = 8 * nt + 2 * tq + (c & 1);
                vals[nt * 4 + c] = (c < 2) ? sum : (sum >> 2); // rows g + 8 were accumulated times 4
                tok[nt * 4 + c] = (token < e.M) ? token : -1;
                row[nt * 4 + c] = u.rb * kTileRows + g + 8 * (c >> 1);
            }
        }
        finish_unit<NT * 4>(e, u, lane, vals, tok, row);
    }
    if (*abort_flag) {
        if (lane == 0) atomicExch(&hdr->status, (int32_t)BITLINEAR_ERR_TIMEOUT);
        // let copies that may still be in flight land before the ring goes away
        const uint64_t t0 = ptx::globaltimer_ns();
        while (ptx::globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
}

// ---------------------------------------------------------------------------------------------
// dp4a path (M <= 8): each lane multiplies its own 2 rows x 32 columns, then the four lanes that share
// a row pair add up with two shuffles.  Kept as an independent cross-check of the MMA path.
__global__ void __launch_bounds__(kWarps * 32) decode_dp4a_kernel(const __grid_constant__ InlineTable inl,
                                                                  const DecodeEntry *__restrict__ table, int n_entries,
                                                                  int total_units, int n_stripes, WorkspaceHeader *hdr)
{
    const DecodeEntry *tab = table ? table : inl.e;
    const int lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3;
    UnitQueue queue;
    queue.init(hdr, (uint32_t)total_units, (uint32_t)n_stripes, blockIdx.x * kWarps + (threadIdx.x >> 5), lane);
    for (;;) {
        const uint32_t unit = queue.next(lane);
        if (unit == 0xFFFFFFFFu) break;
        const int ei = find_entry(tab, n_entries, (int)unit);
        const DecodeEntry &e = tab[ei];
        const UnitCoords u = unit_coords(e, unit);
        const int K = e.K, M = e.M;

        int acc[8][2];
#pragma unroll
        for (int t = 0; t < 8; ++t) acc[t][0] = acc[t][1] = 0;
        const uint4 *wp = e.packed + ((size_t)u.rb * e.KB + u.kt0) * 32 + lane;
        for (int kt = u.kt0; kt < u.kt1; ++kt, wp += 32) {
            const uint4 w = ld_stream(wp);
            const uint32_t words[4] = {w.x, w.y, w.z, w.w};
            const int col = kt * kTileCols + 32 * tq;
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                if (t >= M) break;
                const int8_t *p = e.Xq + (size_t)t * K + col;
                uint4 xa = make_uint4(0u, 0u, 0u, 0u), xb = make_uint4(0u, 0u, 0u, 0u);
                if (col < K) xa = __ldg(reinterpret_cast<const uint4 *>(p));
                if (col + 16 < K) xb = __ldg(reinterpret_cast<const uint4 *>(p + 16));
                const uint32_t xs[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
#pragma unroll
                    for (int f = 0; f < 4; ++f) {
                        const uint32_t codes = (words[i] >> (2 * f)) & 0x03030303u;
                        acc[t][f & 1] = dp4a_u8s8(codes, xs[2 * i + (f >> 1)], acc[t][f & 1]);
                    }
                }
            }
        }
        int vals[16], tok[16], row[16];
#pragma unroll
        for (int t = 0; t < 8; ++t) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                int v = acc[t][h];
                v += __shfl_xor_sync(0xffffffffu, v, 1);
                v += __shfl_xor_sync(0xffffffffu, v, 2);
                vals[2 * t + h] = v;
                tok[2 * t + h] = (t < M && tq == 0) ? t : -1;
                row[2 * t + h] = u.rb * kTileRows + g + 8 * h;
            }
        }
        finish_unit<16>(e, u, lane, vals, tok, row);
    }
}

} // namespace

static int stripes_for(unsigned ctas)
{
    const unsigned warps = ctas * kWarps;
    return (int)(warps < (unsigned)kStripes ? warps : (unsigned)kStripes);
}

template <int NT>
static cudaError_t launch_mma(dim3 grid, dim3 block, const InlineTable &inl, const DecodeEntry *table, int n_entries,
                              int total_units, WorkspaceHeader *hdr, cudaStream_t stream)
{
    static bool attr_set[64] = {false};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(decode_mma_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDecodeSmem);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    decode_mma_kernel<NT><<<grid, block, kDecodeSmem, stream>>>(inl, table, n_entries, total_units, stripes_for(grid.x), hdr);
    return cudaGetLastError();
}

cudaError_t launch_decode(const InlineTable &inl, const DecodeEntry *table, int n_entries, int total_units, int max_M,
                          int path, WorkspaceHeader *hdr, cudaStream_t stream)
{
    if (total_units <= 0) return cudaSuccess;
    int ctas = (total_units + kWarps - 1) / kWarps;
    const dim3 block(kWarps * 32);
    if (path == BITLINEAR_PATH_DP4A) {
        const int cap = sm_count() * 4;
        if (ctas > cap) ctas = cap;
        decode_dp4a_kernel<<<dim3(ctas), block, 0, stream>>>(inl, table, n_entries, total_units, stripes_for(ctas), hdr);
        return cudaGetLastError();
    }
    const int cap = sm_count() * 3; // 3 CTAs x 64 KiB of ring per SM
    if (ctas > cap) ctas = cap;
    const dim3 grid(ctas);
    if (max_M <= 8) return launch_mma<1>(grid, block, inl, table, n_entries, total_units, hdr, stream);
    if (max_M <= 16) return launch_mma<2>(grid, block, inl, table, n_entries, total_units, hdr, stream);
    if (max_M <= 32) return launch_mma<4>(grid, block, inl, table, n_entries, total_units, hdr, stream);
    return launch_mma<8>(grid, block, inl, table, n_entries, total_units, hdr, stream);
}

} // namespace bitlinear
