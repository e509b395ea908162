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

__device__ __forceinline__ uint32_t next_unit(WorkspaceHeader *hdr, int lane)
{
    uint32_t u = 0;
    if (lane == 0) u = atomicAdd(&hdr->unit_counter, 1u);
    return __shfl_sync(0xffffffffu, u, 0);
}

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
template <int NT>
__global__ void __launch_bounds__(kWarps * 32) decode_mma_kernel(const __grid_constant__ InlineTable inl,
                                                                 const DecodeEntry *__restrict__ table, int n_entries,
                                                                 int total_units, WorkspaceHeader *hdr)
{
    const DecodeEntry *tab = table ? table : inl.e;
    const int lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3;
    int ei = 0;
    for (;;) {
        const uint32_t unit = next_unit(hdr, lane);
        if (unit >= (uint32_t)total_units) break;
        while (ei + 1 < n_entries && tab[ei + 1].unit_begin <= (int)unit) ++ei;
        const DecodeEntry &e = tab[ei];
        const UnitCoords u = unit_coords(e, unit);
        const int K = e.K;

        int acc[NT][4];
        const int8_t *xrow[NT];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0;
            const int token = 8 * nt + g; // B-fragment column owned by this lane
            xrow[nt] = (token < e.M) ? e.Xq + (size_t)token * K + 32 * tq : nullptr;
        }
        const uint4 *wp = e.packed + ((size_t)u.rb * e.KB + u.kt0) * 32 + lane;

        for (int kt = u.kt0; kt < u.kt1; kt += kTilesInFlight) {
            uint4 w[kTilesInFlight];
#pragma unroll
            for (int j = 0; j < kTilesInFlight; ++j)
                if (kt + j < u.kt1) w[j] = ld_stream(wp + j * 32);
            wp += kTilesInFlight * 32;
#pragma unroll
            for (int j = 0; j < kTilesInFlight; ++j) {
                if (kt + j >= u.kt1) break;
                const int col = (kt + j) * kTileCols + 32 * tq; // first of this lane's 32 columns
                const uint32_t words[4] = {w[j].x, w[j].y, w[j].z, w[j].w};
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    // activations of columns col .. col+31 of token 8*nt + g; zero beyond K (the padded
                    // weight columns hold code 1, so the activation there must be 0)
                    uint4 xa = make_uint4(0u, 0u, 0u, 0u), xb = make_uint4(0u, 0u, 0u, 0u);
                    if (xrow[nt]) {
                        const int8_t *p = xrow[nt] + (size_t)(kt + j) * kTileCols;
                        if (col < K) xa = __ldg(reinterpret_cast<const uint4 *>(p));
                        if (col + 16 < K) xb = __ldg(reinterpret_cast<const uint4 *>(p + 16));
                    }
                    const uint32_t xs[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint32_t wd = words[i];
                        mma_u8s8(acc[nt], wd & 0x03030303u, (wd >> 2) & 0x03030303u, (wd >> 4) & 0x03030303u,
                                 (wd >> 6) & 0x03030303u, xs[2 * i], xs[2 * i + 1]);
                    }
                }
            }
        }

        // C fragment: c0 (row g, token 2tq), c1 (row g, token 2tq+1), c2 (row g+8, token 2tq), c3 (row g+8, 2tq+1)
        int vals[NT * 4], tok[NT * 4], row[NT * 4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int token = 8 * nt + 2 * tq + (c & 1);
                vals[nt * 4 + c] = acc[nt][c];
                tok[nt * 4 + c] = (token < e.M) ? token : -1;
                row[nt * 4 + c] = u.rb * kTileRows + g + 8 * (c >> 1);
            }
        }
        finish_unit<NT * 4>(e, u, lane, vals, tok, row);
    }
}

// ---------------------------------------------------------------------------------------------
// dp4a path (M <= 8): each lane multiplies its own 2 rows x 32 columns, then the four lanes that share
// a row pair add up with two shuffles.  Kept as an independent cross-check of the MMA path.
__global__ void __launch_bounds__(kWarps * 32) decode_dp4a_kernel(const __grid_constant__ InlineTable inl,
                                                                  const DecodeEntry *__restrict__ table, int n_entries,
                                                                  int total_units, WorkspaceHeader *hdr)
{
    const DecodeEntry *tab = table ? table : inl.e;
    const int lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3;
    int ei = 0;
    for (;;) {
        const uint32_t unit = next_unit(hdr, lane);
        if (unit >= (uint32_t)total_units) break;
        while (ei + 1 < n_entries && tab[ei + 1].unit_begin <= (int)unit) ++ei;
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

cudaError_t launch_decode(const InlineTable &inl, const DecodeEntry *table, int n_entries, int total_units, int max_M,
                          int path, WorkspaceHeader *hdr, cudaStream_t stream)
{
    if (total_units <= 0) return cudaSuccess;
    int ctas = (total_units + kWarps - 1) / kWarps;
    const int cap = sm_count() * 4; // 32 resident warps per SM
    if (ctas > cap) ctas = cap;
    const dim3 grid(ctas), block(kWarps * 32);
    if (path == BITLINEAR_PATH_DP4A) {
        decode_dp4a_kernel<<<grid, block, 0, stream>>>(inl, table, n_entries, total_units, hdr);
    } else if (max_M <= 8) {
        decode_mma_kernel<1><<<grid, block, 0, stream>>>(inl, table, n_entries, total_units, hdr);
    } else if (max_M <= 16) {
        decode_mma_kernel<2><<<grid, block, 0, stream>>>(inl, table, n_entries, total_units, hdr);
    } else if (max_M <= 32) {
        decode_mma_kernel<4><<<grid, block, 0, stream>>>(inl, table, n_entries, total_units, hdr);
    } else {
        decode_mma_kernel<8><<<grid, block, 0, stream>>>(inl, table, n_entries, total_units, hdr);
    }
    return cudaGetLastError();
}

} // namespace bitlinear
