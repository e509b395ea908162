// Kernel (c): weight-streaming ternary x int8 matmul for few tokens (decode): the kernels take up to 64 tokens,
// the library sends them up to 16 (from 17 on the tensor-core GEMM is faster).
//
// The cost of decode is moving the weights from HBM once (Section 1: loading weights from DRAM is
// the expensive part; Section 3: time per output token).  All matrices of a launch form ONE sequence
// of 1 KiB tiles (64 output rows x 64 columns each, row block after row block, matrix after matrix).
// The sequence is split into one equal, contiguous share per warp.  (The kernel can also hold back a part of the
// sequence and cut it into small pieces that the warps draw from a counter when their share is done, so that SMs that
// happen to run faster take more; with the costs of a piece as they are now -- two more row blocks cut and finished by
// the second launch, per piece -- dealing everything statically measured faster on every workload: 68 against 76 us
// on the 7B-shaped up projection set at one token, 75 against 87 us at four, 134 against 138 us on the 3B-shaped
// step, no difference on the 70B-shaped one.  BITLINEAR_DECODE_STATIC_PERCENT below 100 brings the pieces back.)  A warp streams its pieces
// through a private shared-memory ring filled by bulk copies (cp.async.bulk), so the HBM latency is
// covered by the copy engine and not by registers, and the stream never drains at a row-block, matrix
// or piece boundary.  Row blocks that lie completely inside a piece are finished by that warp alone.
// For the row blocks cut by the two ends of a piece the warp only adds its partial sums to an int32
// scratch (fire-and-forget atomics: exact, order-free, nothing to wait for); the warp whose piece reaches
// the END of such a row block notes it in a small list of its own.  A second, very small launch, in which
// one warp takes over the list of one warp of this kernel, dequantises those row blocks.  No flags, no
// scans, no waits between CTAs.
//
// The quantised activations travel the same way.  The quantiser writes them tile by tile ([column tile][token]
// [64 bytes]), so the activations a chunk of weight tiles needs are ONE contiguous range, fetched by a
// second bulk copy into the same ring slot; the B fragments of the MMAs are then conflict-free 16-byte
// shared-memory loads, nothing depends on L1 hit rates when many tokens and many matrices are in flight,
// and columns past K need no special case (the quantiser writes zeros there).
//
// Both launches are programmatic dependents of the launch before them: this kernel starts while the
// activation quantiser is still running and streams weights until it needs the quantiser's outputs; the
// finishing launch is resident, waiting, before this kernel ends.
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
//
// The same kernel streams the base-3 format (five weights per byte, tiles of 80 rows: N*K/5 bytes per matrix).  A
// stored byte is then a number 0..242 and has to be decoded: a table in shared memory (243 entries, one copy per lane
// so that a warp's look-ups never share a bank) turns it into the byte of four 2-bit fields the MMAs above take (rows
// 16 f + r, f = 0..3) plus the code of the fifth row (64 + r), which feeds a fifth MMA as it is.  One look-up per
// stored byte is what this format costs: about 19 instructions per 20 weights where the 2-bit fields cost 3 per 16.
#include <cstdlib>

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
#ifndef BITLINEAR_DECODE_STAGES_NT2
#define BITLINEAR_DECODE_STAGES_NT2 2
#endif
#ifndef BITLINEAR_DECODE_WARPS_NT2
#define BITLINEAR_DECODE_WARPS_NT2 8
#endif
#ifndef BITLINEAR_DECODE_CHUNK_TILES_NT2
#define BITLINEAR_DECODE_CHUNK_TILES_NT2 6
#endif
constexpr int kWarps = BITLINEAR_DECODE_WARPS;             // warps per CTA, each independent
constexpr int kStages = BITLINEAR_DECODE_STAGES;           // chunks in flight per warp
constexpr int kCtasPerSm = BITLINEAR_DECODE_CTAS_PER_SM;
constexpr int kXTileBytes = 64;                            // int8 activations of one token for one column tile

// Shared memory of the kernel for NT 8-token tiles: per warp kStages slots of
// [kTiles weight tiles | kTiles x (up to 8 NT tokens) x 64 bytes of activations], then barriers and a flag.
// (Single-token launches with slots that keep 64 bytes of activations per tile and chunks of 10 to 12 tiles were
// measured: no gain over 8 tiles.  With two token tiles longer chunks do pay: 6 tiles x 2 stages against 4 x 3,
// 104 against 108 us on the 7B-shaped up projection set at 16 tokens.)
template <int NT>
struct Ring {
    static constexpr int kTiles = NT == 1 ? BITLINEAR_DECODE_CHUNK_TILES : (NT == 2 ? BITLINEAR_DECODE_CHUNK_TILES_NT2 : (NT == 8 ? 2 : 4)); // tiles per chunk
    static constexpr int kDepth = NT == 2 ? BITLINEAR_DECODE_STAGES_NT2 : kStages;            // chunks in flight per warp
    static constexpr int kWeightBytes = kTiles * kTileBytes;
    static constexpr int kSlotBytes = kWeightBytes + kTiles * 8 * NT * kXTileBytes;
    static constexpr int kW = NT == 2 ? BITLINEAR_DECODE_WARPS_NT2 : kWarps; // warps per CTA
    static constexpr int kBarsOffset = kW * kDepth * kSlotBytes;
    static constexpr int kAbortOffset = kBarsOffset + kW * kDepth * 8;
    static constexpr int kSmem = kAbortOffset + 16;
    static_assert(kSmem * (NT <= 2 ? kCtasPerSm : 1) <= 227 * 1024, "ring does not fit the SM's shared memory");
    // base-3 format: the decoding table behind the ring, entry v of lane l at 128 v + 4 l
    static constexpr int kLutOffset = (kSmem + 127) / 128 * 128;
    static constexpr int kLutBytes = 243 * 128;
    static constexpr int kSmemTrits = kLutOffset + kLutBytes;
    static_assert(NT != 1 || kSmemTrits <= 227 * 1024, "ring and table do not fit the SM's shared memory");
};
constexpr int kTritRows = 80; // rows of a tile of the base-3 format
#ifndef BITLINEAR_DECODE_STATIC_PERCENT
#define BITLINEAR_DECODE_STATIC_PERCENT 100
#endif
#ifndef BITLINEAR_DECODE_PIECES_PER_WARP
#define BITLINEAR_DECODE_PIECES_PER_WARP 3
#endif
constexpr uint32_t kStaticPercent = BITLINEAR_DECODE_STATIC_PERCENT; // share of the tiles split statically
constexpr uint32_t kPiecesPerWarp = BITLINEAR_DECODE_PIECES_PER_WARP; // dynamic pieces per warp, on average
constexpr uint32_t kMinPieceTiles = 16;
constexpr size_t kStagedTableBytes = 24 * 1024; // see decode_finish_kernel
static_assert(sizeof(DecodeEntry) % 16 == 0, "the table is staged with 16-byte copies");

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

using ptx::bulk_copy_g2s;

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
    return __fdiv_rn(__fmul_rn(*e.gamma, e.beta[token]), e.qb); // (gamma * beta_t) / Qb
}

// What the epilogue needs of a token: its row sum and its scale.  A lane holds outputs of two tokens per 8-token tile
// (2 tq + tb), and it fetches their terms when its warp ENTERS a matrix, not at the end of every row block: there the
// loads (and the division behind them) were a round trip to L2 that the warp sat through before it could store, once
// per token, and a warp that stalls does not catch up with its stream again.
struct TokenTerms {
    int rowsum;
    float scale;
};

template <int NT>
__device__ __forceinline__ void load_terms(const DecodeEntry &e, int tq, TokenTerms (&tt)[NT][2])
{
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
        for (int tb = 0; tb < 2; ++tb) {
            const int token = 8 * nt + 2 * tq + tb;
            tt[nt][tb] = token < e.M ? TokenTerms{e.rowsum[token], token_scale(e, token)} : TokenTerms{0, 0.0f};
        }
    }
}

// End of a row block.  `each(fn)` calls fn(nt, tb, token, row, partial row sum) for every output this lane holds (token
// = 8 nt + 2 tq + tb).  If all KB column tiles went into the sums they are final; otherwise they are added to the
// int32 scratch.
template <int NT, class Each>
__device__ __forceinline__ void finish_block(const DecodeEntry &e, bool complete, const TokenTerms (&tt)[NT][2], Each each)
{
    if (complete)
        each([&](int nt, int tb, int token, int row, int v) { store_result(e, token, row, v, tt[nt][tb].rowsum, tt[nt][tb].scale); });
    else
        each([&](int, int, int token, int row, int v) { atomicAdd(&e.acc32[(size_t)token * e.N + row], v); });
}

// Finishing launch: dequantises the row blocks on one list from the scratch and leaves the scratch clean for
// the next launch.  owned[i] = (entry index, row block).  Up to four row blocks (two with several tokens) are
// handled at a time, and up to four tokens of each, with all loads of one kind issued together, so that the pass
// costs two memory round trips per batch and token group rather than two per row block and token.
// Every list is served by one warp per group of TG tokens (warp (list, group) takes tokens TG * group ..), so that the
// launch takes as long with eight tokens as with one.
// `word` is the lane's 32-bit word of the warp's 128-byte list (one load for the count and all items: every round
// trip of this launch is on the critical path of the step): word 0 the count, words 2 i + 2 and 2 i + 3 item i.
template <int TG, int ROWS> // tokens handled together: 1 (single-token steps), or 4; rows of a row block: 64, or 80
__device__ __forceinline__ void finish_owned_blocks(const DecodeEntry *tab, uint32_t word, int n_owned, int lane, int t0)
{
    // (with static shares a list has at most two row blocks: the two ends of its warp's share)
    constexpr int kBatch = TG == 1 ? 4 : 2;
    constexpr int kParts = (ROWS + 31) / 32; // rows per lane
    for (int b0 = 0; b0 < n_owned; b0 += kBatch) {
        const DecodeEntry *e[kBatch];
        int32_t *acc[kBatch];
        int r0[kBatch], rend[kBatch], N[kBatch], M[kBatch], max_M = 0;
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
            const int item = min(b0 + b, n_owned - 1); // slots past the end repeat the last one and store nothing
            const uint2 o = make_uint2(__shfl_sync(0xffffffffu, word, 2 * item + 2), __shfl_sync(0xffffffffu, word, 2 * item + 3));
            e[b] = tab + o.x;
            r0[b] = (int)o.y * ROWS + lane;
            rend[b] = ((int)o.y + 1) * ROWS;
        }
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
            acc[b] = e[b]->acc32;
            N[b] = (b0 + b < n_owned) ? e[b]->N : 0;
            rend[b] = min(rend[b], N[b]); // rows of this row block that exist
            M[b] = e[b]->M;
            if (N[b] > 0) max_M = max(max_M, M[b]);
        }
        // this warp's TG tokens (t0 ..) of every row block of the batch: all loads first, then all stores
        if (t0 < max_M) {
            int v[kBatch][TG][kParts], rowsum[kBatch][TG];
            float scale[kBatch][TG];
#pragma unroll
            for (int b = 0; b < kBatch; ++b) {
#pragma unroll
                for (int i = 0; i < TG; ++i) {
                    const int t = min(t0 + i, M[b] - 1); // slots past the last token repeat it and store nothing
#pragma unroll
                    for (int h = 0; h < kParts; ++h)
                        v[b][i][h] = (r0[b] + 32 * h < rend[b]) ? __ldcg(acc[b] + (size_t)t * N[b] + r0[b] + 32 * h) : 0;
                    rowsum[b][i] = e[b]->rowsum[t];
                    scale[b][i] = token_scale(*e[b], t);
                }
            }
#pragma unroll
            for (int b = 0; b < kBatch; ++b) {
#pragma unroll
                for (int i = 0; i < TG; ++i) {
                    const int t = t0 + i;
                    if (t >= M[b]) continue;
#pragma unroll
                    for (int h = 0; h < kParts; ++h) {
                        const int r = r0[b] + 32 * h;
                        if (r < rend[b]) {
                            __stcg(acc[b] + (size_t)t * N[b] + r, 0);
                            store_result(*e[b], t, r, v[b][i][h], rowsum[b][i], scale[b][i]);
                        }
                    }
                }
            }
        }
    }
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


// Base-3 format: the four words of a lane's 16 bytes go through the table (entry: bits 0..7 the byte of four 2-bit
// fields, bits 8..9 the fifth code), then four MMAs on the fields as above and a fifth on the fifth codes.
__device__ __forceinline__ void decode_word(uint32_t w, uint32_t lut_lane, uint32_t &fields, uint32_t &fifth)
{
    uint32_t e[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t v = __byte_perm(w, 0u, 0x4440u + i); // byte i, zero-extended
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(e[i]) : "r"(lut_lane + v * 128u));
    }
    const uint32_t t01 = __byte_perm(e[0], e[1], 0x5140u), t23 = __byte_perm(e[2], e[3], 0x5140u);
    fields = __byte_perm(t01, t23, 0x5410u);
    fifth = __byte_perm(t01, t23, 0x7632u);
}

__device__ __forceinline__ void mma_slab_trits(int (&acc)[5][4], const uint4 &stored, uint32_t lut_lane, uint32_t b0, uint32_t b1)
{
    uint4 w, f;
    decode_word(stored.x, lut_lane, w.x, f.x);
    decode_word(stored.y, lut_lane, w.y, f.y);
    decode_word(stored.z, lut_lane, w.z, f.z);
    decode_word(stored.w, lut_lane, w.w, f.w);
    mma_u8s8(acc[0], w.x, w.y, w.z, w.w, b0, b1);
    mma_u8s8(acc[1], w.x & 0xFCFCFCFCu, w.y & 0xFCFCFCFCu, w.z & 0xFCFCFCFCu, w.w & 0xFCFCFCFCu, b0, b1);
    mma_u8s8(acc[2], w.x & 0xF0F0F0F0u, w.y & 0xF0F0F0F0u, w.z & 0xF0F0F0F0u, w.w & 0xF0F0F0F0u, b0, b1);
    mma_u8s8(acc[3], w.x & 0xC0C0C0C0u, w.y & 0xC0C0C0C0u, w.z & 0xC0C0C0C0u, w.w & 0xC0C0C0C0u, b0, b1);
    mma_u8s8(acc[4], f.x, f.y, f.z, f.w, b0, b1);
}

// Un-mixes the four scaled accumulators of every (row, token) this lane holds and hands the row sums to fn.
// C fragment of field f: c0 (row 16f + g, token 2tq), c1 (same row, 2tq + 1), c2 (row 16f + 8 + g, 2tq), c3.
// NF = 5: the base-3 format's fifth accumulator holds the sums of rows 64 + r as they are.
template <int NT, int NF, class Fn>
__device__ __forceinline__ void each_output(const int (&acc)[NT][NF][4], int M, int N, int row0, int tq, Fn fn)
{
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
                const int S[5] = {acc[nt][0][c] - 4 * t1, t1 - 4 * t2, t2 - 4 * t3, t3, acc[nt][NF - 1][c]};
#pragma unroll
                for (int f = 0; f < NF; ++f) {
                    const int r = row0 + 16 * f + 8 * h;
                    if (r < N) fn(nt, tb, token, r, S[f]);
                }
            }
        }
    }
}

// (Two token tiles take 138 registers; held to 128 the kernel was 4 % slower.)
template <int NT, bool kTrits>
__global__ void __launch_bounds__(Ring<NT>::kW * 32, (NT <= 2) ? kCtasPerSm : 1) decode_mma_kernel(
    const __grid_constant__ InlineTable inl, const DecodeEntry *__restrict__ table, int n_entries,
    uint32_t total_tiles, uint32_t share, uint32_t dyn, WorkspaceHeader *hdr, OwnedList *lists, const WaitHooks hooks)
{
    extern __shared__ __align__(128) uint8_t dsmem[];
    ptx::griddep_launch_dependents(); // the finishing launch may become resident; it waits for this grid to end
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3;
    using R = Ring<NT>;
    constexpr int kChunkTiles = R::kTiles;
    constexpr int kStages = R::kDepth; // (the ring depth of this form)
    const uint32_t ring = ptx::smem_u32(dsmem) + warp * (kStages * R::kSlotBytes);
    const uint32_t bars = ptx::smem_u32(dsmem + R::kBarsOffset) + warp * (kStages * 8);
    int n_owned = 0;
    volatile int *abort_flag = reinterpret_cast<volatile int *>(dsmem + R::kAbortOffset);

    constexpr int kFields = kTrits ? 5 : 4, kRows = kTrits ? kTritRows : kTileRows;
    const uint32_t lut_lane = ptx::smem_u32(dsmem + R::kLutOffset) + lane * 4;
    if (kTrits) {
        // entry v of every lane's copy: the byte of four 2-bit fields c0 + 4 c1 + 16 c2 + 64 c3, and c4 << 8
        uint32_t *lut = reinterpret_cast<uint32_t *>(dsmem + R::kLutOffset);
        for (int v = threadIdx.x; v < 243; v += R::kW * 32) {
            const uint32_t c0 = v % 3, c1 = (v / 3) % 3, c2 = (v / 9) % 3, c3 = (v / 27) % 3, c4 = v / 81;
            const uint32_t entry = c0 | (c1 << 2) | (c2 << 4) | (c3 << 6) | (c4 << 8);
            for (int l = 0; l < 32; ++l) lut[v * 32 + l] = entry;
        }
    }
    if (threadIdx.x == 0) *abort_flag = 0;
    if (lane == 0) {
        // two arrivals per phase: one announces the weight bytes of a chunk, one its activation bytes
#pragma unroll
        for (int s = 0; s < kStages; ++s) ptx::mbar_init(bars + 8 * s, 2);
        ptx::fence_mbar_init();
    }
    __syncthreads();

    const DecodeEntry *tab = table ? table : inl.e;

    // A piece is a contiguous range of the tile sequence.  Piece w (w < n_warps) is warp w's own share of
    // `share` tiles; the tiles after the shares form pieces of `dyn` tiles dealt through hdr->piece_counter.
    const uint32_t n_warps = gridDim.x * R::kW, w = blockIdx.x * R::kW + warp;
    uint2 *owned = lists[w].item;
    struct Piece {
        const DecodeEntry *e;
        int rb, kt, left; // first tile (row block, column tile) and number of tiles; left == 0: no piece
    };
    auto locate = [&](uint32_t t_begin, uint32_t t_end) {
        Piece p;
        p.e = tab + find_entry(tab, n_entries, t_begin, lane);
        const uint32_t local = t_begin - p.e->tile_begin, kb = (uint32_t)p.e->KB;
        p.rb = (int)(local / kb);
        p.kt = (int)(local - (uint32_t)p.rb * kb);
        p.left = (int)(t_end - t_begin);
        return p;
    };
    uint32_t drawn = 0;        // lane 0: result of the draw in flight
    bool drawing = dyn != 0;   // a draw is in flight
    auto draw = [&]() {
        if (lane == 0) drawn = atomicAdd(&hdr->piece_counter, 1u);
    };
    // The next dynamic piece (none: left == 0); normally leaves another draw in flight.  Every piece in hand can
    // add one row block to the warp's list, so a warp whose list is nearly full stops drawing BEFORE it
    // claims another piece; the number of pieces is far too small for every warp to get there.
    auto next_piece = [&]() {
        Piece p;
        p.e = tab;
        p.rb = p.kt = p.left = 0;
        if (!drawing) return p;
        drawing = false;
        const uint64_t t0 = (uint64_t)share * n_warps + (uint64_t)__shfl_sync(0xffffffffu, drawn, 0) * dyn;
        if (t0 >= total_tiles) return p;
        if (n_owned + 3 <= kMaxOwned) {
            draw();
            drawing = true;
        }
        const uint64_t t1 = t0 + dyn;
        return locate((uint32_t)t0, (uint32_t)(t1 < total_tiles ? t1 : total_tiles));
    };

    // ---- streaming phase (a lambda, so that a warp without work can leave it early)
    [&]() {

    // Two cursors walk the pieces: the producer issues copies up to kStages chunks ahead of the consumer and
    // may already be in the next piece.  A chunk is up to kChunkTiles tiles and never crosses the end of a
    // row block, so both cursors cut a piece into the same chunks.
    Piece cur, nxt;
    {
        // own share, clipped to the sequence (without a dynamic part the shares are rounded up)
        const uint64_t s0 = (uint64_t)w * share, s1 = s0 + share;
        const uint32_t lim = dyn ? share * n_warps : total_tiles;
        if (s0 >= lim) { // no share (small launches): nothing to stream ahead of the wait
            ptx::griddep_wait();
            return;
        }
        cur = locate((uint32_t)s0, (uint32_t)(s1 < lim ? s1 : lim));
    }
    nxt = cur;
    nxt.left = 0;            // the first dynamic piece is drawn below, after the first copies have been issued,
    bool nxt_pending = false; // and looked at only when a cursor gets to the end of `cur`
    auto resolve_next = [&]() {
        if (nxt_pending) {
            nxt_pending = false;
            nxt = next_piece();
        }
    };

    const DecodeEntry *pe;   // producer: matrix, tiles left in the piece, place in the row block,
    int p_left, p_kt, p_KB, p_blocks; // row blocks left in the matrix (this one included)
    const uint8_t *p_src;
    const int8_t *p_x; // the matrix's activations, [column tile][token][64 bytes]
    int p_xbytes;      // activation bytes per column tile = tokens * 64
    bool p_on_next = false;  // producer already works on `nxt`
    auto producer_start = [&](const Piece &p) {
        pe = p.e;
        p_left = p.left;
        p_kt = p.kt;
        p_KB = p.e->KB;
        p_blocks = p.e->NB - p.rb;
        p_src = reinterpret_cast<const uint8_t *>(p.e->packed) + ((size_t)p.rb * p_KB + p.kt) * kTileBytes;
        p_x = p.e->Xq;
        p_xbytes = p.e->M * kXTileBytes;
    };
    producer_start(cur);
    uint32_t issued = 0, consumed = 0; // chunks, over the whole kernel (ring slot = count % kStages)

    // Activation copies must not be issued before the quantiser's results are visible; the weight copies of
    // the first chunks are.  The activation copies of those chunks are kept here and issued after the wait.
    bool x_ready = false;
    const int8_t *held_x[kStages];
    uint32_t held_bytes[kStages];
    int n_held = 0;

    auto top_up = [&]() {
        while (issued - consumed < (uint32_t)kStages) {
            if (p_left == 0) {
                resolve_next();
                if (p_on_next || nxt.left == 0) break;
                producer_start(nxt);
                p_on_next = true;
            }
            const int n = min(min(kChunkTiles, p_KB - p_kt), p_left);
            const uint32_t s = issued % kStages;
            const int8_t *xsrc = p_x + (size_t)p_kt * p_xbytes;
            const uint32_t xbytes = (uint32_t)(n * p_xbytes);
            if (lane == 0) {
                const uint32_t slot = ring + s * R::kSlotBytes;
                ptx::mbar_arrive_expect_tx(bars + 8 * s, (uint32_t)n * kTileBytes);
                bulk_copy_g2s(slot, p_src, (uint32_t)n * kTileBytes, bars + 8 * s);
                if (x_ready) {
                    ptx::mbar_arrive_expect_tx(bars + 8 * s, xbytes);
                    bulk_copy_g2s(slot + R::kWeightBytes, xsrc, xbytes, bars + 8 * s);
                }
            }
            if (!x_ready) { // at most kStages chunks are issued before the wait, into slots 0, 1, ...
                held_x[n_held] = xsrc;
                held_bytes[n_held] = xbytes;
                ++n_held;
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
                    p_x = pe->Xq;
                    p_xbytes = pe->M * kXTileBytes;
                }
            }
        }
    };
    top_up();
    // The weights above are never written by a kernel.  Everything below (the header's counters, the
    // quantised activations, their scales and sums, the scratch) is written by the launch before this one:
    // when this kernel was launched ahead of that launch's end, wait for it here.
    ptx::griddep_wait();
    x_ready = true;
    if (lane == 0) {
#pragma unroll
        for (int i = 0; i < kStages; ++i) {
            if (i < n_held) {
                // (test device: the first warp of the launch leaves out the arrival that announces its first chunk's
                // activation bytes, and the copy it announces with it: the phase never completes)
                if (hooks.skip_arrive && w == 0 && i == 0) continue;
                ptx::mbar_arrive_expect_tx(bars + 8 * i, held_bytes[i]);
                bulk_copy_g2s(ring + i * R::kSlotBytes + R::kWeightBytes, held_x[i], held_bytes[i], bars + 8 * i);
            }
        }
    }
    if (drawing) {
        draw();
        nxt_pending = true;
    }

    // consumer
    const DecodeEntry *e = cur.e;
    int KB = e->KB, rb = cur.rb, kt = cur.kt, left = cur.left;
    TokenTerms terms[NT][2];
    load_terms<NT>(*e, tq, terms);

    bool alive = true;
    while (alive) {
        if (left == 0) { // piece done: go on with the next one, which the producer has normally begun already
            resolve_next();
            if (nxt.left == 0) break;
            if (!p_on_next) producer_start(nxt);
            p_on_next = false;
            if (nxt.e != e) load_terms<NT>(*nxt.e, tq, terms);
            e = nxt.e;
            KB = e->KB;
            rb = nxt.rb;
            kt = nxt.kt;
            left = nxt.left;
            nxt = next_piece();
            top_up();
        }
        // ---- one row block (or the part of it that lies in this piece)
        const int M = e->M;
        int acc[NT][kFields][4]; // [token tile][field][C fragment]
        uint32_t xlane[NT]; // offset of this lane's B-fragment token (lanes without a token read the last one) and columns
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
            for (int f = 0; f < kFields; ++f) acc[nt][f][0] = acc[nt][f][1] = acc[nt][f][2] = acc[nt][f][3] = 0;
            xlane[nt] = (uint32_t)(R::kWeightBytes + min(8 * nt + g, M - 1) * kXTileBytes + 16 * tq);
        }
        const uint32_t xtile = (uint32_t)(M * kXTileBytes); // activation bytes per column tile in the slot
        int tiles = 0; // tiles of this row block accumulated here
        while (kt < KB && left > 0) {
            const int n = min(min(kChunkTiles, KB - kt), left);
            const uint32_t s = consumed % kStages;
            const uint32_t slot = ring + s * R::kSlotBytes;
            if (!ptx::mbar_wait_bounded(bars + 8 * s, (consumed / kStages) & 1u, abort_flag, hooks.limit_us)) { alive = false; break; }
            // (n is the same for all lanes: mma.sync needs the whole warp)
            if (n == kChunkTiles) {
#pragma unroll
                for (int t = 0; t < kChunkTiles; ++t) {
                    const uint4 w0 = lds128(slot + t * kTileBytes + lane * 16);
                    const uint4 w1 = lds128(slot + t * kTileBytes + 512 + lane * 16);
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        const uint4 x = lds128(slot + t * xtile + xlane[nt]);
                        if constexpr (kTrits) {
                            mma_slab_trits(acc[nt], w0, lut_lane, x.x, x.y);
                            mma_slab_trits(acc[nt], w1, lut_lane, x.z, x.w);
                        } else {
                            mma_slab(acc[nt], w0, x.x, x.y);
                            mma_slab(acc[nt], w1, x.z, x.w);
                        }
                    }
                }
            } else {
#pragma unroll
                for (int t = 0; t < kChunkTiles; ++t) {
                    if (t < n) {
                        const uint4 w0 = lds128(slot + t * kTileBytes + lane * 16);
                        const uint4 w1 = lds128(slot + t * kTileBytes + 512 + lane * 16);
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            const uint4 x = lds128(slot + t * xtile + xlane[nt]);
                            if constexpr (kTrits) {
                                mma_slab_trits(acc[nt], w0, lut_lane, x.x, x.y);
                                mma_slab_trits(acc[nt], w1, lut_lane, x.z, x.w);
                            } else {
                                mma_slab(acc[nt], w0, x.x, x.y);
                                mma_slab(acc[nt], w1, x.z, x.w);
                            }
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

        // A row block of which only a part was summed here goes through the scratch; the warp that reaches
        // its end dequantises it in the final pass.
        const bool complete = tiles == KB;
        if (!complete && kt == KB) {
            if (lane == 0) owned[n_owned] = make_uint2((uint32_t)(e - tab), (uint32_t)rb);
            ++n_owned; // cannot exceed kMaxOwned: see next_piece
        }
        finish_block<NT>(*e, complete, terms, [&](auto fn) { each_output<NT, kFields>(acc, M, e->N, rb * kRows + g, tq, fn); });

        // next row block, or next matrix
        if (kt == KB) {
            kt = 0;
            if (++rb == e->NB && left > 0) {
                ++e;
                rb = 0;
                KB = e->KB;
                load_terms<NT>(*e, tq, terms);
            }
        }
    }
    }();

    if (*abort_flag) {
        if (lane == 0) atomicExch(&hdr->status, (int32_t)BITLINEAR_ERR_TIMEOUT);
        // let copies that may still be in flight land before the ring goes away
        const uint64_t t0 = ptx::globaltimer_ns();
        while (ptx::globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    }

    if (lane == 0) lists[w].n = (uint32_t)n_owned;
}

// ---------------------------------------------------------------------------------------------
// The same matmul for 13 to 64 tokens: 13 to 16 tokens when a launch streams 1.5 GB of weights or more (see
// decode_is_wide: the kernel above with two token tiles per warp is faster on shorter launches, 104 against 122 us on the
// 7B-shaped up projection set at 16 tokens, and slower on the 70B-shaped step), 17 to 64 tokens through the test hook
// only (the library sends those to the tensor-core GEMM).  With many tokens the activations of a chunk are as large as, or
// larger than, its weights, so here the eight warps of a CTA share them: the CTA walks a
// sequence of GROUP tiles (one row block per warp x one column tile), warp i streams row block warps * group + i
// through its own ring exactly as above, and the activations of a chunk are fetched ONCE per CTA into a
// shared ring.  Two barriers per activation slot keep the warps together: `xfull` (the copy has landed) and
// `xempty` (all eight warps are done with the slot; only then does warp 0 refill it), so the warps of a CTA
// are never more than the ring depth apart.  The CTAs take equal contiguous shares of the group-tile
// sequence; cut row blocks go through the scratch and the per-warp lists as above.
template <int NT>
struct WideRing {
    static constexpr int kW = decode_wide_warps(8 * NT);           // warps per CTA = row blocks per group tile
    static constexpr int kTiles = NT == 2 ? 8 : (NT == 4 ? 6 : 4); // column tiles per chunk
    static constexpr int kDepth = NT == 8 ? 4 : 3;                  // chunks in flight
    static constexpr int kWeightBytes = kTiles * kTileBytes;
    static constexpr int kXSlotBytes = kTiles * 8 * NT * kXTileBytes;
    static constexpr int kXOffset = kW * kDepth * kWeightBytes;
    static constexpr int kBarsOffset = kXOffset + kDepth * kXSlotBytes;
    static constexpr int kAbortOffset = kBarsOffset + (kW + 2) * kDepth * 8;
    static constexpr int kSmem = kAbortOffset + 16;
    static_assert(kSmem <= 227 * 1024, "rings do not fit the SM's shared memory");
};

template <int NT>
__global__ void __launch_bounds__(WideRing<NT>::kW * 32, 1) decode_wide_kernel(
    const __grid_constant__ InlineTable inl, const DecodeEntry *__restrict__ table, int n_entries,
    uint32_t total_items, uint32_t share, WorkspaceHeader *hdr, OwnedList *lists, const WaitHooks hooks)
{
    extern __shared__ __align__(128) uint8_t dsmem[];
    ptx::griddep_launch_dependents();
    using R = WideRing<NT>;
    constexpr int kChunkTiles = R::kTiles, kDepth = R::kDepth, kW = R::kW;
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3;
    const uint32_t wring = ptx::smem_u32(dsmem) + warp * (kDepth * R::kWeightBytes);
    const uint32_t xring = ptx::smem_u32(dsmem + R::kXOffset);
    const uint32_t wbars = ptx::smem_u32(dsmem + R::kBarsOffset) + warp * (kDepth * 8); // this warp's weights have landed
    const uint32_t xfull = ptx::smem_u32(dsmem + R::kBarsOffset) + kW * kDepth * 8; // the CTA's activations have landed
    const uint32_t xempty = xfull + kDepth * 8;                                         // all warps are done with them
    volatile int *abort_flag = reinterpret_cast<volatile int *>(dsmem + R::kAbortOffset);
    const uint32_t w = blockIdx.x * kW + warp;
    uint2 *owned = lists[w].item;
    int n_owned = 0;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
#pragma unroll
        for (int s = 0; s < kDepth; ++s) {
            ptx::mbar_init(xfull + 8 * s, 1);
            ptx::mbar_init(xempty + 8 * s, kW);
        }
    }
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < kDepth; ++s) ptx::mbar_init(wbars + 8 * s, 1);
        ptx::fence_mbar_init();
    }
    __syncthreads();

    const DecodeEntry *tab = table ? table : inl.e;
    const uint64_t i0 = (uint64_t)blockIdx.x * share;
    const uint32_t i1 = (uint32_t)(i0 + share < total_items ? i0 + share : total_items);

    // A walker steps through the CTA's share chunk by chunk; producer and consumer each have one.
    struct Walker {
        const DecodeEntry *e;
        int KB, groups, group, kt, left;
    };
    struct Chunk {
        const DecodeEntry *e;
        int group, kt, n;
        bool ends_group;
    };
    auto step = [](Walker &p) {
        Chunk c;
        c.e = p.e;
        c.group = p.group;
        c.kt = p.kt;
        c.n = min(min(kChunkTiles, p.KB - p.kt), p.left);
        p.kt += c.n;
        p.left -= c.n;
        c.ends_group = p.kt == p.KB;
        if (c.ends_group) {
            p.kt = 0;
            if (++p.group == p.groups && p.left > 0) {
                ++p.e;
                p.KB = p.e->KB;
                p.groups = (p.e->NB + kW - 1) / kW;
                p.group = 0;
            }
        }
        return c;
    };

    [&]() {
    if (i0 >= i1) {
        ptx::griddep_wait();
        return;
    }
    Walker prod;
    prod.e = tab + find_entry(tab, n_entries, (uint32_t)i0, lane);
    prod.KB = prod.e->KB;
    prod.groups = (prod.e->NB + kW - 1) / kW;
    {
        const uint32_t local = (uint32_t)i0 - prod.e->tile_begin;
        prod.group = (int)(local / (uint32_t)prod.KB);
        prod.kt = (int)(local - (uint32_t)prod.group * (uint32_t)prod.KB);
    }
    prod.left = (int)(i1 - (uint32_t)i0);
    Walker cons = prod;
    uint32_t issued = 0, consumed = 0;

    bool x_ready = false; // see the kernel above: activation copies wait for the launch before this one
    const int8_t *held_x[kDepth];
    uint32_t held_bytes[kDepth];
    int n_held = 0;
    bool alive = true;

    auto top_up = [&]() {
        while (alive && prod.left > 0 && issued - consumed < (uint32_t)kDepth) {
            const uint32_t s = issued % kDepth;
            if (warp == 0 && issued >= (uint32_t)kDepth) {
                // the slot's previous contents must have been consumed by all eight warps
                if (!ptx::mbar_wait_bounded(xempty + 8 * s, (issued / kDepth - 1) & 1u, abort_flag, hooks.limit_us)) {
                    alive = false;
                    break;
                }
            }
            const Chunk c = step(prod);
            const int rb = c.group * kW + warp;
            const int xb = c.e->M * kXTileBytes;
            const int8_t *xsrc = c.e->Xq + (size_t)c.kt * xb;
            const uint32_t xbytes = (uint32_t)(c.n * xb);
            if (lane == 0) {
                if (rb < c.e->NB) {
                    const uint8_t *src = reinterpret_cast<const uint8_t *>(c.e->packed) + ((size_t)rb * c.e->KB + c.kt) * kTileBytes;
                    ptx::mbar_arrive_expect_tx(wbars + 8 * s, (uint32_t)c.n * kTileBytes);
                    bulk_copy_g2s(wring + s * R::kWeightBytes, src, (uint32_t)c.n * kTileBytes, wbars + 8 * s);
                } else {
                    ptx::mbar_arrive(wbars + 8 * s); // no row block for this warp: the slot's phase still has to advance
                }
                if (warp == 0 && x_ready) {
                    ptx::mbar_arrive_expect_tx(xfull + 8 * s, xbytes);
                    bulk_copy_g2s(xring + s * R::kXSlotBytes, xsrc, xbytes, xfull + 8 * s);
                }
            }
            if (!x_ready) {
                held_x[n_held] = xsrc;
                held_bytes[n_held] = xbytes;
                ++n_held;
            }
            ++issued;
        }
    };
    top_up();
    ptx::griddep_wait();
    x_ready = true;
    if (warp == 0 && lane == 0) {
#pragma unroll
        for (int i = 0; i < kDepth; ++i) {
            if (i < n_held) {
                // (test device: the first CTA leaves out the arrival that announces its first activation chunk, and
                // the copy it announces with it)
                if (hooks.skip_arrive && blockIdx.x == 0 && i == 0) continue;
                ptx::mbar_arrive_expect_tx(xfull + 8 * i, held_bytes[i]);
                bulk_copy_g2s(xring + i * R::kXSlotBytes, held_x[i], held_bytes[i], xfull + 8 * i);
            }
        }
    }

    const DecodeEntry *terms_of = nullptr; // the matrix whose token terms this lane holds
    TokenTerms terms[NT][2];
    while (alive && cons.left > 0) {
        // ---- one group of row blocks (or the part of it that lies in this share); this warp's row block is rb
        const DecodeEntry *e = cons.e;
        if (e != terms_of) {
            load_terms<NT>(*e, tq, terms);
            terms_of = e;
        }
        const int M = e->M, KB = cons.KB;
        const int rb = cons.group * kW + warp;
        const bool active = rb < e->NB; // the last group of a matrix may have fewer than eight row blocks
        int acc[NT][4][4];
        uint32_t xlane[NT];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
            for (int f = 0; f < 4; ++f) acc[nt][f][0] = acc[nt][f][1] = acc[nt][f][2] = acc[nt][f][3] = 0;
            xlane[nt] = (uint32_t)(min(8 * nt + g, M - 1) * kXTileBytes + 16 * tq);
        }
        const uint32_t xtile = (uint32_t)(M * kXTileBytes);
        int tiles = 0;
        bool ended = false;
        while (!ended && cons.left > 0) {
            const Chunk c = step(cons);
            ended = c.ends_group;
            const uint32_t s = consumed % kDepth;
            const uint32_t parity = (consumed / kDepth) & 1u;
            if (!ptx::mbar_wait_bounded(xfull + 8 * s, parity, abort_flag, hooks.limit_us) ||
                (active && !ptx::mbar_wait_bounded(wbars + 8 * s, parity, abort_flag, hooks.limit_us))) {
                alive = false;
                break;
            }
            if (active) { // (the same for all lanes: mma.sync needs the whole warp)
                const uint32_t wslot = wring + s * R::kWeightBytes + lane * 16;
                const uint32_t xslot = xring + s * R::kXSlotBytes;
#pragma unroll
                for (int t = 0; t < kChunkTiles; ++t) {
                    if (t < c.n) {
                        const uint4 w0 = lds128(wslot + t * kTileBytes);
                        const uint4 w1 = lds128(wslot + t * kTileBytes + 512);
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            const uint4 x = lds128(xslot + t * xtile + xlane[nt]);
                            mma_slab(acc[nt], w0, x.x, x.y);
                            mma_slab(acc[nt], w1, x.z, x.w);
                        }
                    }
                }
            }
            __syncwarp(); // every lane has read both slots
            if (lane == 0) ptx::mbar_arrive(xempty + 8 * s);
            ++consumed;
            tiles += c.n;
            top_up();
        }
        if (!alive) break;
        if (active) {
            const bool complete = tiles == KB;
            if (!complete && ended) {
                if (n_owned < kMaxOwned) {
                    if (lane == 0) owned[n_owned] = make_uint2((uint32_t)(e - tab), (uint32_t)rb);
                    ++n_owned;
                }
            }
            finish_block<NT>(*e, complete, terms, [&](auto fn) { each_output<NT, 4>(acc, M, e->N, rb * kTileRows + g, tq, fn); });
        }
    }
    }();

    if (*abort_flag) {
        if (lane == 0) atomicExch(&hdr->status, (int32_t)BITLINEAR_ERR_TIMEOUT);
        const uint64_t t0 = ptx::globaltimer_ns();
        while (ptx::globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    if (lane == 0) lists[w].n = (uint32_t)n_owned;
}

// The finishing launch: warp w takes the list of warp w of the kernel above.
// staged_entries > 0: the CTA copies that many entries of the table (all of them) into its shared memory while the
// matmul is still running, which takes the table's round trip to L2 off the chain list -> entry -> sums -> stores.
// (One instance per form, so that each takes only the registers it needs: beside a CTA of the matmul an SM has room
// for a finishing CTA of at most 130 registers per thread, and a finishing CTA that is not resident, waiting, when the
// matmul ends costs the step several microseconds.)
template <int TG, int ROWS>
__global__ void __launch_bounds__(256, 2) decode_finish_kernel(const __grid_constant__ InlineTable inl,
                                                               const DecodeEntry *__restrict__ table,
                                                               const OwnedList *__restrict__ lists, uint32_t n_lists,
                                                               int staged_entries, int token_groups)
{
    extern __shared__ uint4 staged_table[];
    // warp (list w, token group tg)
    const uint32_t gw = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const uint32_t groups = (uint32_t)token_groups;
    const uint32_t w = gw / groups;
    const int t0 = (int)(gw - w * groups) * TG;
    // The quantiser of a step that follows may become resident at once; it waits for this grid to end before it
    // touches anything, and the matmul behind it streams weights (never written) until that quantiser has ended.
    ptx::griddep_launch_dependents();
    if (staged_entries > 0) { // (the table is written once, when the sequence is created)
        const int n_vec = staged_entries * (int)(sizeof(DecodeEntry) / 16);
        const uint4 *src = reinterpret_cast<const uint4 *>(table);
        for (int i = threadIdx.x; i < n_vec; i += blockDim.x) staged_table[i] = __ldg(src + i);
        __syncthreads();
        table = reinterpret_cast<const DecodeEntry *>(staged_table);
    }
    ptx::griddep_wait(); // the lists and the scratch are written by the launch before this one
    if (w >= n_lists) return;
    const int lane = threadIdx.x & 31;
    const uint32_t word = __ldcg(reinterpret_cast<const uint32_t *>(&lists[w]) + lane);
    const int n = (int)__shfl_sync(0xffffffffu, word, 0);
    if (n == 0) return;
    finish_owned_blocks<TG, ROWS>(table ? table : inl.e, word, n, lane, t0);
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
    const int M = e.M, KB = e.KB;
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
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                if (t >= M) break;
                const uint4 xa = __ldg(reinterpret_cast<const uint4 *>(e.Xq + ((size_t)kt * M + t) * kXTileBytes + 16 * tq));
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

// Measurement aid, compiled in only with -DBITLINEAR_TUNING (the library as built by build.py reads no environment
// variable): a positive integer in the environment overrides a tuning constant.
static uint32_t tuning_from_env(const char *name, uint32_t fallback, uint32_t max_value)
{
#ifdef BITLINEAR_TUNING
    const char *v = std::getenv(name);
    if (!v || !*v) return fallback;
    const long x = std::atol(v);
    return (x >= 1 && x <= (long)max_value) ? (uint32_t)x : fallback;
#else
    (void)name;
    (void)max_value;
    return fallback;
#endif
}

// Launches `kernel` as a programmatic dependent of the launch before it in the stream (it may start early and
// must wait, on the device, before it reads what that launch writes).  early == false: an ordinary launch.
static cudaError_t launch_dependent(const void *kernel, dim3 grid, dim3 block, size_t smem, void **args, bool early,
                                    cudaStream_t stream)
{
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cfg.attrs = &attr;
    cfg.numAttrs = early ? 1 : 0;
    return cudaLaunchKernelExC(&cfg, kernel, args);
}

// Launches the finishing kernel for n_lists lists of a launch whose largest token count is max_M.
static cudaError_t launch_finish(const InlineTable &inl, const DecodeEntry *table, const OwnedList *lists, uint32_t n_lists,
                                 int staged, int max_M, bool trits, bool early, cudaStream_t stream)
{
    const bool single = max_M == 1;
    int token_groups = single ? 1 : (max_M + 3) / 4; // warps per list
    const void *kernel = trits ? (single ? (const void *)decode_finish_kernel<1, kTritRows> : (const void *)decode_finish_kernel<4, kTritRows>)
                               : (single ? (const void *)decode_finish_kernel<1, kTileRows> : (const void *)decode_finish_kernel<4, kTileRows>);
    void *fargs[] = {(void *)&inl, (void *)&table, (void *)&lists, (void *)&n_lists, (void *)&staged, (void *)&token_groups};
    const uint32_t finish_warps = n_lists * (uint32_t)token_groups;
    return launch_dependent(kernel, dim3((finish_warps + 7) / 8), dim3(256), (size_t)staged * sizeof(DecodeEntry), fargs, early,
                            stream);
}

template <int NT, bool kTrits>
static cudaError_t launch_mma(dim3 grid, dim3 block, const InlineTable &inl, const DecodeEntry *table, int n_entries,
                              uint32_t total_tiles, uint32_t share, uint32_t dyn, int max_M, WorkspaceHeader *hdr,
                              OwnedList *lists, cudaStream_t stream)
{
    WaitHooks hooks = take_wait_hooks();

    constexpr int kSmemBytes = kTrits ? Ring<NT>::kSmemTrits : Ring<NT>::kSmem;
    static bool attr_set[64] = {false};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(decode_mma_kernel<NT, kTrits>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    static const bool early = tuning_from_env("BITLINEAR_DECODE_EARLY_LAUNCH", 1, 2) == 1; // 2 = off
    void *args[] = {(void *)&inl, (void *)&table, (void *)&n_entries, (void *)&total_tiles, (void *)&share,
                    (void *)&dyn, (void *)&hdr, (void *)&lists, (void *)&hooks};
    cudaError_t err = launch_dependent((const void *)decode_mma_kernel<NT, kTrits>, grid, block, kSmemBytes, args, early, stream);
    if (err != cudaSuccess) return err;
    uint32_t n_lists = grid.x * Ring<NT>::kW;
    // a table that fits beside the matmul's ring (one CTA of each per SM) is staged in the finishing CTAs' shared memory
    // (the base-3 form's decoding table takes that room: its finishing CTAs read the table from global memory)
    int staged = (!kTrits && table && (size_t)n_entries * sizeof(DecodeEntry) <= kStagedTableBytes) ? n_entries : 0;
    return launch_finish(inl, table, lists, n_lists, staged, max_M, kTrits, early, stream);
}

template <int NT>
static cudaError_t launch_wide(dim3 grid, dim3 block, const InlineTable &inl, const DecodeEntry *table, int n_entries,
                               uint32_t total_items, uint32_t share, int max_M, WorkspaceHeader *hdr, OwnedList *lists,
                               cudaStream_t stream)
{
    WaitHooks hooks = take_wait_hooks();
    static bool attr_set[64] = {false};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(decode_wide_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, WideRing<NT>::kSmem);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    static const bool early = tuning_from_env("BITLINEAR_DECODE_EARLY_LAUNCH", 1, 2) == 1; // 2 = off
    void *args[] = {(void *)&inl, (void *)&table, (void *)&n_entries, (void *)&total_items, (void *)&share,
                    (void *)&hdr, (void *)&lists, (void *)&hooks};
    cudaError_t err = launch_dependent((const void *)decode_wide_kernel<NT>, grid, block, WideRing<NT>::kSmem, args, early, stream);
    if (err != cudaSuccess) return err;
    uint32_t n_lists = grid.x * WideRing<NT>::kW;
    int staged = 0; // (this kernel's rings leave no room beside them)
    return launch_finish(inl, table, lists, n_lists, staged, max_M, false, early, stream);
}

cudaError_t launch_decode(const InlineTable &inl, const DecodeEntry *table, int n_entries, uint32_t total_tiles,
                          int max_M, int path, WorkspaceHeader *hdr, OwnedList *lists, cudaStream_t stream, bool trits, bool wide)
{
    if (total_tiles == 0) return cudaSuccess;
    if (trits && (max_M > 8 || path == BITLINEAR_PATH_DP4A)) return cudaErrorInvalidValue;
    const dim3 block(kWarps * 32);
    if (max_M > 16) wide = true; // (beyond 16 tokens only the lockstep kernel exists)
    if (path != BITLINEAR_PATH_DP4A && wide && !trits) {
        // total_tiles counts group tiles here; one CTA per SM, equal contiguous shares, at least 4 items each
        const uint32_t warps = (uint32_t)decode_wide_warps(max_M);
        uint32_t ctas = (total_tiles + 3) / 4;
        uint32_t cap = (uint32_t)sm_count();
        if (cap > kMaxDecodeWarps / warps) cap = kMaxDecodeWarps / warps;
        if (ctas > cap) ctas = cap;
        const uint32_t share = (total_tiles + ctas - 1) / ctas;
        const dim3 grid(ctas), wide_block(warps * 32);
        if (max_M <= 16) return launch_wide<2>(grid, wide_block, inl, table, n_entries, total_tiles, share, max_M, hdr, lists, stream);
        if (max_M <= 32) return launch_wide<4>(grid, wide_block, inl, table, n_entries, total_tiles, share, max_M, hdr, lists, stream);
        return launch_wide<8>(grid, wide_block, inl, table, n_entries, total_tiles, share, max_M, hdr, lists, stream);
    }
    if (path == BITLINEAR_PATH_DP4A) {
        int ctas = (inl.e[0].NB + kWarps - 1) / kWarps;
        const int cap = sm_count() * 4;
        if (ctas > cap) ctas = cap;
        decode_dp4a_kernel<<<dim3(ctas), block, 0, stream>>>(inl);
        return cudaGetLastError();
    }
    // every warp should have at least kMinTilesPerWarp tiles; beyond that, fill the machine
    constexpr uint32_t kMinTilesPerWarp = 4;
    const uint32_t warps = (max_M > 8 && !trits) ? (uint32_t)Ring<2>::kW : (uint32_t)kWarps;
    uint32_t ctas = (total_tiles + kMinTilesPerWarp * warps - 1) / (kMinTilesPerWarp * warps);
    uint32_t cap = (uint32_t)sm_count() * kCtasPerSm;
    if (cap > kMaxDecodeWarps / warps) cap = kMaxDecodeWarps / warps;
    if (ctas > cap) ctas = cap;
    const dim3 grid(ctas);
    // Static shares take kStaticPercent of the tiles; the rest is dealt in pieces of `dyn` tiles, about
    // kPiecesPerWarp per warp, none shorter than kMinPieceTiles.  Small launches have no dynamic part.
    static const uint32_t static_percent = tuning_from_env("BITLINEAR_DECODE_STATIC_PERCENT", kStaticPercent, 100);
    static const uint32_t pieces_per_warp = tuning_from_env("BITLINEAR_DECODE_PIECES_PER_WARP", kPiecesPerWarp, 8);
    const uint32_t n_warps = ctas * warps;
    uint32_t share = total_tiles / n_warps, dyn = 0;
    if (share >= 4 * kMinPieceTiles && static_percent < 100) {
        share = (uint32_t)((uint64_t)total_tiles * static_percent / 100 / n_warps);
        if (share == 0) share = 1; // (a warp without a share never draws a piece)
        const uint32_t rest = total_tiles - share * n_warps;
        dyn = rest / (n_warps * pieces_per_warp);
        if (dyn < kMinPieceTiles) dyn = kMinPieceTiles;
    } else {
        share = (total_tiles + n_warps - 1) / n_warps; // all static: the last warps may get less, or nothing
    }
    if (trits) return launch_mma<1, true>(grid, block, inl, table, n_entries, total_tiles, share, dyn, max_M, hdr, lists, stream);
    if (max_M > 8) return launch_mma<2, false>(grid, dim3(warps * 32), inl, table, n_entries, total_tiles, share, dyn, max_M, hdr, lists, stream);
    return launch_mma<1, false>(grid, block, inl, table, n_entries, total_tiles, share, dyn, max_M, hdr, lists, stream);
}

} // namespace bitlinear
