// Kernel (d): ternary x int8 GEMM for 65 tokens and more on the tcgen05 tensor cores (17 to 64 tokens: decode_tc.cu,
// which this file's launchers hand those launches to).
//
// With hundreds of tokens every weight is reused hundreds of times, so the integer matmul
// (Section 1 / Section 3 "Energy": matrix multiplication dominates) is a dense contraction and
// belongs on the tensor cores; from 65 to 128 tokens the same kernel streams the weights faster than the
// warp-level MMAs of the decode kernel can.  Per CTA tile of 128 tokens x 256 output features, per 128-wide
// k block:
//   producer warp  : TMA loads the int8 activation tile (128 x 128 B, 128-byte swizzle) and the
//                    packed 2-bit weight tiles (4 row blocks x 2 column tiles x 1 KiB) into shared memory;
//   expander warps : turn the 2-bit codes into unsigned bytes with ONE mask per four weights -- the field
//                    of row 16 f + r stays where it is, so the byte is code * 4^f -- and write them
//                    K-major with the same 128-byte swizzle the tensor core expects;
//   MMA thread     : issues four tcgen05.mma kind::i8 (128 x 256 x 32, s8 x u8) per k block into a TMEM
//                    accumulator; one tcgen05.commit releases the TMA stage and the expanded tile;
//   epilogue warps : tcgen05.ld the finished int32 accumulators, undo the 4^f of their output row with an
//                    exact shift, subtract the token's sum of q (codes are T + 1), scale by
//                    gamma * beta_t / 127, round to bf16 and store, while the MMA warp fills the second
//                    TMEM buffer.  |acc| <= 64 * 2 * 127 * K < 2^31 for every K the library accepts.
// With more than 128 tokens a CTA takes TWO token tiles per feature tile (MT = 2): the expanded weight
// tile, the costly operand (written once and read once per MMA through shared memory, whose bandwidth bounds
// this kernel), then feeds two MMAs per k step, and the two accumulators fill the tensor memory, so the
// epilogue of a tile no longer overlaps the next tile's MMAs.
// One launch runs one matmul (passed as a kernel parameter) or all the matmuls of a sequence (a table in device
// memory): the CTAs walk one launch-wide sequence of CTA tiles.  When whole tiles would leave many SMs idle in the
// last round (160 tiles on 148 SMs), the launch instead gives every CTA an equal, contiguous share of the sequence of
// K BLOCKS of all tiles: a CTA's share then begins and ends inside tiles, the tile it begins in is finished by the CTA
// in front of it, and partial sums travel through a scratch slot per CTA (see Schedule below).  With at most half as many
// tiles as SMs every tile is split along K among several CTAs, each of which then finishes its part of the tile's outputs
// (split_factor below).
// The kernel is a programmatic dependent of the activation quantiser: set-up (barriers, tensor memory,
// descriptor prefetch) runs while the quantiser finishes; the producer waits for it before the first load.
// All waits are bounded; on expiry the CTA sets the workspace status to BITLINEAR_ERR_TIMEOUT,
// every role leaves its loop, TMEM is released and the kernel returns.
//
// Roofline: int8 tensor throughput; algorithmic work 2*M*N*K integer operations.
#include <cuda.h>

#include <cstdlib>
#include <cstring>

#include "gemm_problem.cuh"
#include "internal.cuh"
#include "ptx.cuh"
#include "tma_host.cuh"

namespace bitlinear {

namespace {

using namespace ptx;

// BM = 128 tokens per MMA (MMA M, TMEM lanes), BN = 256 features per tile (MMA N, TMEM columns per accumulator),
// BK = 128 bytes of K per stage: gemm_problem.cuh
constexpr int kMaxStages = 12; // ring of TMA stages (activations + packed weights); its depth is chosen at launch
constexpr int kMaxBSlots = 3;  // ring of expanded weight tiles (its depth: Cfg)
constexpr int kTmemCols = 512;
constexpr int kFetchBufs = 6;  // see Schedule below

constexpr int kProducerWarp = 0;
constexpr int kMmaWarp = 1;
// warps 2..5 are the epilogue (one per TMEM lane quarter)
constexpr int kFirstExpanderWarp = 6; // 8 warps
constexpr int kExpanderWarps = 8;
constexpr int kThreads = (kFirstExpanderWarp + kExpanderWarps) * 32; // 448

constexpr uint32_t kBBytes = BN * BK;            // 32 KiB expanded weights
constexpr uint32_t kPBytes = (BN / kTileRows) * (BK / kTileCols) * kTileBytes; //  8 KiB packed weights

// Expanding one k block takes a warp about 700 cycles from the stage's arrival to the hand-over (two waits, 32 KiB
// of stores that all eight warps push through shared memory at once, a proxy fence of about 300 cycles), whatever
// the number of warps that share it.  With two token tiles the MMAs of a k block take longer than that.  With one
// they take 512 cycles, so there the expander warps form two groups that take k blocks in turn (each warp two
// packed tiles of every other k block), with a third expanded tile so that both groups can be ahead of the MMAs.
template <int MT>
struct Cfg {
    static constexpr int kAccBufs = (MT == 1) ? 2 : 1; // MT * BN * kAccBufs = all 512 TMEM columns
    static constexpr int kGroups = (MT == 1) ? 2 : 1;  // expander groups
    static constexpr int kBSlots = (MT == 1) ? 3 : 2;  // expanded weight tiles
};

// Shared memory: [expanded weight tiles: 2 or 3 x 32 KiB][TMA stages: n x (activations | 8 KiB packed)][barriers].
// What waits on memory (the TMA stages) and what the expander hands to the tensor core (the expanded tiles)
// have rings of their own: the expanded tile is four times the packed one, and with one ring the 227 KiB held
// three or four k blocks in flight, too few to cover the latency of HBM when the weights are streamed once
// (few tokens).  A stage's activation part is a_rows = 128 rows of 128 bytes per token tile (launches whose largest M
// is 64 or less ask for 64 rows and go to the weight-stationary kernel of decode_tc.cu instead).
constexpr uint32_t kSmemLimit = 232448; // 227 KiB
constexpr uint32_t kBarrierBytes = 512;
__host__ __device__ constexpr uint32_t stage_bytes(int mt, int a_rows) { return (uint32_t)(mt * a_rows * BK) + kPBytes; }
inline int b_slots(int mt) { return mt == 1 ? Cfg<1>::kBSlots : Cfg<2>::kBSlots; }
inline int stages_that_fit(int mt, int a_rows)
{
    const int n = (int)((kSmemLimit - 1024 /*alignment slack*/ - kBarrierBytes - b_slots(mt) * kBBytes) / stage_bytes(mt, a_rows));
    return n < kMaxStages ? n : kMaxStages;
}
inline uint32_t smem_bytes_for(int mt, int a_rows, int n_stages)
{
    return 1024 + b_slots(mt) * kBBytes + (uint32_t)n_stages * stage_bytes(mt, a_rows) + kBarrierBytes;
}

struct Barriers {
    uint64_t full[kMaxStages];   // TMA bytes landed (activations + packed weights)
    uint64_t empty[kMaxStages];  // MMAs that read the stage have completed
    uint64_t expanded[kMaxBSlots]; // int8 weight tile written
    uint64_t acc_full[2];        // accumulator(s) of a tile complete
    uint64_t acc_empty[2];       // drained by the epilogue
    uint64_t epilogue_met;       // rendezvous of the four epilogue warps (after a contribution)
    uint64_t last_full;          // the accumulators of the CTA's last unit are complete (for the warps that only help there)
    uint64_t fetched[4][kFetchBufs]; // finisher: a piece of a contribution has landed in an epilogue warp's buffer
    uint32_t tmem_base;
    int abort_flag;
};
static_assert(sizeof(Barriers) <= kBarrierBytes, "barrier block");

// How the work of a launch is dealt to its CTAs.
//   whole tiles : CTA b takes CTA tiles b, b + grid, b + 2 grid, ...
//   k-block shares (stream_k): the k blocks of all tiles form one sequence of total_kb items, and CTA b takes the
//     contiguous range [b * total_kb / grid, (b + 1) * total_kb / grid), which it cuts at tile borders into units.  A
//     unit that covers its whole tile is an ordinary tile.  A unit that begins inside its tile (it can only be the
//     CTA's first) is a CONTRIBUTION: the CTA writes its int32 partial sums to its own scratch slot with plain stores
//     and then sets its flag.  A unit that begins with the tile but ends inside it (it can only be the CTA's last) makes
//     the CTA the tile's FINISHER: the rest of the tile belongs to the first units of the CTAs behind it (b + 1 .. the
//     CTA that holds the tile's last k block), which were those CTAs' first work and are long done; the finisher waits
//     for their flags (a bounded wait), adds their slots to its own sums and dequantises.  No CTA ever waits for work
//     that itself waits, flags must be zero when the launch starts, slots need no clearing.
//   split tiles (stream_k == 2): tile t belongs to CTAs s t .. s t + s - 1, each with 1/s of its k blocks (its only
//     unit) and 1/s of its outputs to finish: see split_factor.
struct Schedule {
    int stream_k; // 0: whole tiles, 1: k-block shares, 2: split tiles
    int split;    // split tiles: CTAs per tile
    int n_tiles;
    long long total_kb;
    uint32_t *flags; // one word per CTA
    int32_t *slots;  // per CTA: [token tile][lane quarter][chunk of 32 features][lane][32 sums]
};
constexpr uint32_t kSlotTileBytes = BM * BN * 4; // partial sums of one token tile of a CTA tile
constexpr size_t kFlagBytes = 1024;              // flags in front of the slots (one word per CTA)
// The finisher fetches contributions with bulk copies into shared memory (its rings are idle by then: a finisher unit
// is its CTA's last), kFetchBufs pieces of kFetchBytes in flight per epilogue warp: reading them with plain loads would
// be one round trip to L2 after the other (measured: 1.2 us each, 16 per contribution).
constexpr uint32_t kFetchChunks = 2;                    // chunks of 32 features per piece
constexpr uint32_t kFetchBytes = kFetchChunks * 4096;   // 8 KiB
static_assert(4 * kFetchBufs * kFetchBytes <= 3 * 64 * 1024, "the fetch buffers lie inside the idle rings");

// Byte offset of 16-byte piece `piece` (of 8) of lane `lane` inside a chunk of 32 lanes x 128 bytes: piece-major, so that
// the 32 lanes of a warp write (global memory) and read (shared memory, after the bulk copy) 512 consecutive bytes per
// instruction -- four full lines per store (lane-major rows made every store instruction touch 32 lines, 16 bytes of
// each), no bank conflicts per load.  The slots in global memory have this layout (they reach shared memory by bulk
// copies, as they are).
__device__ __forceinline__ uint32_t slot_piece(int lane, int piece) { return (uint32_t)(piece * 512 + lane * 16); }

enum UnitKind { kWholeTile = 0, kContribution = 1, kFinisher = 2, kSplit = 3 };

struct Unit {
    int tile, kb0, kb1, kind;
    int last_contributor; // finisher: the contributions are the first units of CTAs blockIdx.x + 1 .. last_contributor
    int split_s, split_r; // split tile: the tile belongs to split_s CTAs, this one is number split_r of them
};

// Position in the ring of TMA stages and in the ring of expanded tiles after `it` k blocks.
struct RingPos {
    int s;          // TMA stage
    uint32_t round; // times the TMA ring has been gone through
    uint32_t it;    // k blocks so far: expanded-tile slot it % slots, use it / slots
    __device__ RingPos() : s(0), round(0), it(0) {}
    __device__ void advance(int n_stages)
    {
        ++it;
        if (++s == n_stages) {
            s = 0;
            ++round;
        }
    }
};

// Steps through the units of this CTA.  Every role of the CTA runs its own walker; all of them see the same units.
template <bool kTable>
struct UnitWalker {
    const Schedule &sc;
    ProblemCursor<kTable> cur;
    int next_tile;        // whole tiles
    long long pos, end;   // k-block shares
    __device__ UnitWalker(const Schedule &sc_, const GemmProblem &one, const GemmProblem *t, int n)
        : sc(sc_), cur(one, t, n), next_tile((int)blockIdx.x), pos(0), end(0)
    {
        if (sc.stream_k == 1) {
            pos = (long long)blockIdx.x * sc.total_kb / (long long)gridDim.x;
            end = (long long)(blockIdx.x + 1) * sc.total_kb / (long long)gridDim.x;
        }
    }
    // whether another unit follows the one `next` returned last
    __device__ bool more() const
    {
        if (sc.stream_k == 2) return false;
        return sc.stream_k ? pos < end : next_tile < sc.n_tiles;
    }
    // the next unit and its matmul; false: none is left
    __device__ bool next(Unit &u, const GemmProblem *&g)
    {
        u.split_s = 1;
        u.split_r = 0;
        if (sc.stream_k == 2) { // split tiles: CTA b is number b % s of the s CTAs of tile b / s, its only unit
            if (next_tile < 0) return false;
            const int s = sc.split;
            u.tile = (int)blockIdx.x / s;
            u.split_s = s;
            u.split_r = (int)blockIdx.x % s;
            g = &cur.seek(u.tile);
            const int KB = g->p.KB;
            u.kb0 = (int)((long long)u.split_r * KB / s);
            u.kb1 = (int)((long long)(u.split_r + 1) * KB / s);
            u.kind = kSplit;
            u.last_contributor = 0;
            next_tile = -1;
            return true;
        }
        if (!sc.stream_k) {
            if (next_tile >= sc.n_tiles) return false;
            g = &cur.seek(next_tile);
            u.tile = next_tile;
            u.kb0 = 0;
            u.kb1 = g->p.KB;
            u.kind = kWholeTile;
            u.last_contributor = 0;
            next_tile += (int)gridDim.x;
            return true;
        }
        if (pos >= end) return false;
        g = &cur.seek_kb(pos);
        const int KB = g->p.KB;
        const long long local = pos - g->p.kb_begin;
        const int tile_local = (int)(local / KB);
        u.tile = g->p.tile_begin + tile_local;
        u.kb0 = (int)(local - (long long)tile_local * KB);
        const long long tile_start = pos - u.kb0, tile_end = tile_start + KB;
        u.kb1 = (int)((end < tile_end ? end : tile_end) - tile_start);
        u.last_contributor = 0;
        if (u.kb0 > 0) {
            u.kind = kContribution;
        } else if (u.kb1 < KB) {
            u.kind = kFinisher;
            // the CTA whose range holds the tile's last k block: the largest c with c * total_kb / grid <= tile_end - 1
            u.last_contributor = (int)((tile_end * (long long)gridDim.x - 1) / sc.total_kb);
        } else {
            u.kind = kWholeTile;
        }
        pos = tile_start + u.kb1;
        return true;
    }
};

// Shift, subtract, scale, round and store the 32 sums `v` of chunk c (features n0 + 32 c ..) of token t.
__device__ __forceinline__ void emit_chunk(const Params &p, int n0, const uint32_t (&v)[32], int c, int t, int rowsum, float scale)
{
    const int n = n0 + c * 32;
    // output row n + i carries the factor 4^f, f = ((n + i) % 64) / 16 = 2 (c % 2) + i / 16
    const int sh_lo = 4 * (c & 1), sh_hi = sh_lo + 2;
    int a[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) a[i] = ((int)v[i] >> (i < 16 ? sh_lo : sh_hi)) - rowsum;
    if (t >= p.M) return;
    if (p.out_i32) {
        int32_t *dst = reinterpret_cast<int32_t *>(p.out) + (size_t)t * p.N + n;
#pragma unroll
        for (int i = 0; i < 32; i += 4)
            if (n + i < p.N) *reinterpret_cast<int4 *>(dst + i) = make_int4(a[i], a[i + 1], a[i + 2], a[i + 3]);
    } else {
        __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(p.out) + (size_t)t * p.N + n;
#pragma unroll
        for (int i = 0; i < 32; i += 16) { // N is a multiple of 16: 16 features are in or out together
            if (n + i < p.N) {
                uint32_t o[8];
#pragma unroll
                for (int h = 0; h < 8; ++h) {
                    const float x0 = __fmul_rn((float)a[i + 2 * h], scale);
                    const float x1 = __fmul_rn((float)a[i + 2 * h + 1], scale);
                    const __nv_bfloat162 pr = __floats2bfloat162_rn(x0, x1);
                    o[h] = *reinterpret_cast<const uint32_t *>(&pr);
                }
                if (p.out_32b_aligned) {
                    st_global_v8(dst + i, o);
                } else {
                    *reinterpret_cast<uint4 *>(dst + i) = make_uint4(o[0], o[1], o[2], o[3]);
                    *reinterpret_cast<uint4 *>(dst + i + 8) = make_uint4(o[4], o[5], o[6], o[7]);
                }
            }
        }
    }
}

// The sum of q and the scale gamma * beta_t / Q_b of token t (past M: zeros).
__device__ __forceinline__ void token_terms(const Params &p, float gamma, int t, int &rowsum, float &scale)
{
    rowsum = 0;
    scale = 0.0f;
    if (t < p.M) {
        rowsum = p.rowsum[t];
        if (!p.out_i32) scale = __fdiv_rn(__fmul_rn(gamma, p.beta[t]), p.qb);
    }
}

// Jobs first, first + step, ... of a tile whose sums are complete in tensor memory (nothing to add): this warp's lane
// quarter q of (token tile, pair of 32-feature chunks).  The epilogue warps run this for every whole tile; for the last
// tile of a CTA, whose epilogue nothing overlaps, the two expander warps of the same lane quarter take two thirds of the jobs.
template <int MT>
__device__ __forceinline__ void finish_whole_jobs(const Params &p, uint32_t tmem_base, int q, int lane, int buf, int m0, int n0,
                                                  int halves, int first, int step)
{
    constexpr int kPairs = BN / 32 / (int)kFetchChunks;
    const float gamma = p.out_i32 ? 0.0f : *p.gamma;
#pragma unroll 1
    for (int jb = first; jb < halves * kPairs; jb += step) {
        const int half = jb / kPairs, c0 = (jb % kPairs) * (int)kFetchChunks;
        const uint32_t acc_col = (uint32_t)((buf * MT + half) * BN);
        const int t = m0 + half * BM + 32 * q + lane;
        int rowsum;
        float scale;
        token_terms(p, gamma, t, rowsum, scale);
        uint32_t v[kFetchChunks][32];
#pragma unroll
        for (int cc = 0; cc < (int)kFetchChunks; ++cc)
            tmem_ld_32x32(tmem_base + ((uint32_t)(32 * q) << 16) + acc_col + (uint32_t)((c0 + cc) * 32), v[cc]);
        tmem_ld_wait();
#pragma unroll
        for (int cc = 0; cc < (int)kFetchChunks; ++cc) emit_chunk(p, n0, v[cc], c0 + cc, t, rowsum, scale);
    }
}

template <int MT, bool kTable>
__global__ void __launch_bounds__(kThreads, 1)
prefill_gemm_kernel(const __grid_constant__ GemmProblem one, const GemmProblem *__restrict__ table, int n_problems,
                    const Schedule sc, int a_rows, int n_stages, const WaitHooks hooks)
{
    constexpr int kAccBufs = Cfg<MT>::kAccBufs, kBSlots = Cfg<MT>::kBSlots, kGroups = Cfg<MT>::kGroups;
    const uint32_t kStageBytes = stage_bytes(MT, a_rows), kAHalfBytes = (uint32_t)(a_rows * BK);
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u; // swizzled tiles need 1024-byte alignment
    uint8_t *smem = smem_raw + (base - raw);
    const uint32_t stages = base + kBSlots * kBBytes; // first TMA stage
    Barriers *bars = reinterpret_cast<Barriers *>(smem + kBSlots * kBBytes + (uint32_t)n_stages * kStageBytes);
    volatile int *abort_flag = &bars->abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(smem_u32(&bars->full[s]), 1);
            mbar_init(smem_u32(&bars->empty[s]), 1);
        }
        for (int b = 0; b < kBSlots; ++b) {
            mbar_init(smem_u32(&bars->expanded[b]), kExpanderWarps / kGroups);
        }
        for (int b = 0; b < kAccBufs; ++b) {
            mbar_init(smem_u32(&bars->acc_full[b]), 1);
            mbar_init(smem_u32(&bars->acc_empty[b]), 4);
        }
        mbar_init(smem_u32(&bars->epilogue_met), 4);
        mbar_init(smem_u32(&bars->last_full), 1);
        for (int w = 0; w < 4; ++w)
            for (int b = 0; b < kFetchBufs; ++b) mbar_init(smem_u32(&bars->fetched[w][b]), 1);
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

    int32_t *const status = kTable ? table[0].p.status : one.p.status; // (the same for every matmul of a launch)

    if (warp == kProducerWarp) {
        if (lane == 0) {
            UnitWalker<kTable> walk(sc, one, table, n_problems);
            if (!kTable) {
                prefetch_tensormap(&one.tmap_x);
                prefetch_tensormap(&one.tmap_w);
            }
            griddep_wait(); // the activations are written by the launch before this one
            RingPos pos;
            bool ok = true;
            Unit unit;
            const GemmProblem *gp;
            while (ok && walk.next(unit, gp)) {
                const GemmProblem &g = *gp;
                const Params &p = g.p;
                const int local = unit.tile - p.tile_begin;
                const int m0 = (local % p.tiles_m) * (MT * BM);
                const int n0 = (local / p.tiles_m) * BN;
                const int halves = (MT == 2 && m0 + BM < p.M) ? 2 : 1; // a second token tile past the end is left out
                for (int kb = unit.kb0; kb < unit.kb1; ++kb, pos.advance(n_stages)) {
                    const int s = pos.s;
                    if (pos.round > 0 && !mbar_wait_bounded(smem_u32(&bars->empty[s]), (pos.round - 1) & 1, abort_flag, hooks.limit_us)) {
                        ok = false;
                        break;
                    }
                    const uint32_t full = smem_u32(&bars->full[s]);
                    const uint32_t a_dst = stages + s * kStageBytes;
                    const uint32_t p_dst = a_dst + MT * kAHalfBytes;
                    // (test device: the first CTA leaves out the arrival that announces its first stage's bytes, and
                    // the loads it announces with it, so that nothing is in flight for a phase that never completes)
                    if (hooks.skip_arrive && blockIdx.x == 0 && pos.it == 0) continue;
                    mbar_arrive_expect_tx(full, halves * kAHalfBytes + kPBytes);
                    tma_load_2d(a_dst, &g.tmap_x, kb * BK, m0, full);       // x = byte column (multiple of 128)
                    if (halves == 2) tma_load_2d(a_dst + kAHalfBytes, &g.tmap_x, kb * BK, m0 + BM, full);
                    tma_load_3d(p_dst, &g.tmap_w, 0, kb * (BK / kTileCols), n0 / kTileRows, full); // x = 0: whole tiles
                }
            }
        }
    } else if (warp == kMmaWarp) {
        // ONE thread runs this loop.  What it executes per k block (a wait, the MMAs, a commit: 60 to 90 cycles
        // each on B200) is serial, and the tensor core idles whenever that takes longer than the MMAs themselves,
        // so there is one wait and one commit per k block: `expanded` implies `full` (the expander warps waited for
        // the stage before they arrived), and `empty` also tells the expander that the expanded tile was read.
        if (lane == 0) {
            const uint32_t idesc = idesc_i8(BM, BN, /*a_signed=*/1, /*b_signed=*/0);
            UnitWalker<kTable> walk(sc, one, table, n_problems);
            uint32_t tile_it = 0;
            bool ok = true;
            // The thread's own instructions are on the critical path too, so nothing is recomputed per k block: the
            // low words of the operand descriptors (address / 16) and the barrier addresses of the ring positions
            // advance by constants, the high word of the descriptors never changes.
            const uint32_t desc_hi = (uint32_t)(smem_desc_k_sw128(0) >> 32);
            auto desc = [&](uint32_t lo) { return ((uint64_t)desc_hi << 32) | lo; };
            const uint32_t a_lo0 = (uint32_t)smem_desc_k_sw128(stages), a_step = kStageBytes >> 4, a_half = kAHalfBytes >> 4;
            const uint32_t b_lo0 = (uint32_t)smem_desc_k_sw128(base), b_step = kBBytes >> 4;
            const uint32_t empty0 = smem_u32(&bars->empty[0]), expanded0 = smem_u32(&bars->expanded[0]);
            uint32_t s = 0, b = 0, b_parity = 0; // TMA stage; expanded tile and the parity of its use
            uint32_t a_lo = a_lo0, b_lo = b_lo0, empty_bar = empty0, expanded_bar = expanded0;
            Unit unit;
            const GemmProblem *gp;
            for (; ok && walk.next(unit, gp); ++tile_it) {
                const int tile = unit.tile;
                const Params &p = gp->p;
                const int kb_begin = unit.kb0, kb_end = unit.kb1;
                const int buf = tile_it % kAccBufs;
                const uint32_t use = tile_it / kAccBufs;
                if (use > 0 && !mbar_wait_bounded(smem_u32(&bars->acc_empty[buf]), (use - 1) & 1, abort_flag, hooks.limit_us)) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * MT * BN);
                const bool two = MT == 2 && ((tile - p.tile_begin) % p.tiles_m) * (MT * BM) + BM < p.M;
                uint32_t accumulate = 0;
                for (int kb = kb_begin; kb < kb_end; ++kb) {
                    if (!mbar_wait_bounded(expanded_bar, b_parity, abort_flag, hooks.limit_us)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
#pragma unroll
                    for (int k4 = 0; k4 < BK / 32; ++k4) { // 32 bytes of K = 2 descriptor units further
                        const uint64_t b_desc = desc(b_lo + 2 * k4);
                        mma_i8_ss(d_tmem, desc(a_lo + 2 * k4), b_desc, idesc, accumulate);
                        if (two) mma_i8_ss(d_tmem + BN, desc(a_lo + a_half + 2 * k4), b_desc, idesc, accumulate);
                        accumulate = 1;
                    }
                    mma_commit(empty_bar); // stage and expanded tile are reusable once these MMAs have read them
                    if (++s == (uint32_t)n_stages) {
                        s = 0;
                        a_lo = a_lo0;
                        empty_bar = empty0;
                    } else {
                        a_lo += a_step;
                        empty_bar += 8;
                    }
                    if (++b == (uint32_t)kBSlots) {
                        b = 0;
                        b_lo = b_lo0;
                        expanded_bar = expanded0;
                        b_parity ^= 1u;
                    } else {
                        b_lo += b_step;
                        expanded_bar += 8;
                    }
                }
                if (ok) mma_commit(smem_u32(&bars->acc_full[buf]));
                if (ok && !walk.more()) mma_commit(smem_u32(&bars->last_full));
            }
        }
    } else if (warp >= kFirstExpanderWarp) {
        // An expander warp owns packed tile (row block rbi, column tile kti) of the stage: warp ew tile
        // (ew / 2, ew % 2) of every k block, or, in two groups, warp ew tiles (ew % 4, 0) and (ew % 4, 1) of the k
        // blocks with it % 2 == ew / 4.  The 16 bytes
        // at slot 4 g + tq of each slab hold the codes of rows 16 f + 8 h + g at columns
        // 16 tq + 8 s + 4 hi + b (slab s, word 2 hi + h, byte b, field f): 16 consecutive columns of a row
        // are words (h, 2 + h) of slab 0 followed by words (h, 2 + h) of slab 1.
        // Which thread takes which slot is free here.  Eight consecutive threads take g in {q, (q ^ 1) + 4}
        // (q = lane / 8) and tq = 0..3: their 16-byte loads fall into eight different bank groups, and so do
        // their 16-byte stores, because the swizzled chunk (4 kti + tq) ^ g then takes eight different values.
        const int ew = warp - kFirstExpanderWarp;
        const int q = lane >> 3;
        const int g = (lane & 4) ? ((q ^ 1) + 4) : q, tq = lane & 3;
        const int slot = 4 * g + tq;
        const int group = (kGroups == 2) ? (ew >> 2) : 0;
        const int rbi = (kGroups == 2) ? (ew & 3) : (ew >> 1);
        UnitWalker<kTable> walk(sc, one, table, n_problems);
        RingPos pos, reader; // reader: the k block kBSlots steps back, whose MMAs read the expanded tile written next
        bool ok = true;
        Unit unit;
        const GemmProblem *gp = nullptr;
        uint32_t n_units = 0;
        while (ok && walk.next(unit, gp)) {
            ++n_units;
            const int kb_end = unit.kb1;
            for (int kb = unit.kb0; kb < kb_end; ++kb, pos.advance(n_stages)) {
                const int s = pos.s, b = (int)(pos.it % kBSlots);
                const bool mine = kGroups == 1 || (int)(pos.it & 1u) == group;
                const bool has_reader = pos.it >= (uint32_t)kBSlots;
                const int rs = reader.s;
                const uint32_t rround = reader.round;
                if (has_reader) reader.advance(n_stages);
                if (!mine) continue;
                if (!mbar_wait_bounded(smem_u32(&bars->full[s]), pos.round & 1, abort_flag, hooks.limit_us)) {
                    ok = false;
                    break;
                }
                // (the reader's stage is not refilled before this tile is expanded: its `empty` phase is the latest)
                if (has_reader && !mbar_wait_bounded(smem_u32(&bars->empty[rs]), rround & 1, abort_flag, hooks.limit_us)) {
                    ok = false;
                    break;
                }
                const uint8_t *stage = smem + kBSlots * kBBytes + s * kStageBytes;
                uint8_t *bt = smem + b * kBBytes;
#pragma unroll
                for (int kk = 0; kk < kGroups; ++kk) { // the packed tiles of this warp
                    const int kti = (kGroups == 2) ? kk : (ew & 1);
                    const uint4 *packed =
                        reinterpret_cast<const uint4 *>(stage + MT * kAHalfBytes) + (rbi * 2 + kti) * (kTileBytes / 16);
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
                }
                fence_proxy_async_smem(); // generic-proxy writes -> visible to the tensor core
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars->expanded[b]));
            }
        }
        // The CTA's last unit, when it is a whole tile: this warp takes a third of the jobs of its lane quarter (see the
        // epilogue warps below, which take the jobs 0, 3, 6, ...).
        if (ok && n_units > 0 && unit.kind == kWholeTile) {
            const Params &p = gp->p;
            const int local = unit.tile - p.tile_begin;
            const int m0 = (local % p.tiles_m) * (MT * BM), n0 = (local / p.tiles_m) * BN;
            const int halves = (MT == 2 && m0 + BM < p.M) ? 2 : 1;
            const int buf = (int)((n_units - 1) % kAccBufs);
            // (not `acc_full`: this warp may be several tiles ahead of the MMAs, and a wait on a phase's parity only
            // works for a waiter that is at most one phase behind)
            if (mbar_wait_bounded(smem_u32(&bars->last_full), 0, abort_flag, hooks.limit_us)) {
                tc_fence_after_sync();
                finish_whole_jobs<MT>(p, tmem_base, warp & 3, lane, buf, m0, n0, halves, 1 + (ew >> 2), 3);
            }
        }
    } else {
        // epilogue: warp w may touch TMEM lanes 32*(w % 4) .. +31
        const int q = warp & 3;
        UnitWalker<kTable> walk(sc, one, table, n_problems);
        uint32_t tile_it = 0;
        Unit unit;
        const GemmProblem *gp;
        for (; walk.next(unit, gp); ++tile_it) {
            const int tile = unit.tile;
            const Params &p = gp->p;
            const float gamma = p.out_i32 ? 0.0f : *p.gamma;
            const int local = tile - p.tile_begin;
            const int m0 = (local % p.tiles_m) * (MT * BM);
            const int n0 = (local / p.tiles_m) * BN;
            const int buf = tile_it % kAccBufs;
            const uint32_t parity = (tile_it / kAccBufs) & 1;
            const int halves = (MT == 2 && m0 + BM < p.M) ? 2 : 1; // no MMA wrote the accumulator of an absent token tile
            if (!mbar_wait_bounded(smem_u32(&bars->acc_full[buf]), parity, abort_flag, hooks.limit_us)) break;
            tc_fence_after_sync();

            // the token whose sums this thread's TMEM lane holds (past M: none)
            auto token_of_lane = [&](int half) {
                return m0 + half * BM + 32 * q + lane;
            };
            // the 4 KiB that hold this warp's 32 x 32 sums of chunk c of token tile `half` in the slot of CTA `cta` (the
            // chunks of a warp follow each other)
            auto slot_chunk = [&](int cta, int half, int c) {
                return reinterpret_cast<uint8_t *>(sc.slots) + (size_t)cta * (MT * kSlotTileBytes) +
                       (size_t)((half * 4 + q) * (BN / 32) + c) * 4096;
            };

            // The sums of a tile are handled as jobs: (token tile, pair of chunks of 32 features), this warp's lane quarter
            // of each.  A whole tile: the CTA finishes all jobs, nothing to fetch.  A contribution: all jobs go to the
            // CTA's slot.  A finisher: all jobs, with the slots of the CTAs behind it added.  A split tile: the CTA
            // finishes the jobs r, r + s, ... with the slots of the other CTAs of its tile added, and writes the rest.
            constexpr int kPairs = BN / 32 / (int)kFetchChunks;
            const int n_jobs_tile = halves * kPairs;
            const bool split = unit.kind == kSplit;
            // (the last unit of the CTA, when it is a whole tile: the two expander warps of this lane quarter, idle by then,
            // take the jobs 1, 4, 7, ... and 2, 5, 8, ...: nothing overlaps this epilogue)
            const bool shared_last = unit.kind == kWholeTile && !walk.more();
            const int job_start = split ? unit.split_r : 0, job_stride = split ? unit.split_s : (shared_last ? 3 : 1);
            const int n_contrib = unit.kind == kFinisher ? unit.last_contributor - (int)blockIdx.x : (split ? unit.split_s - 1 : 0);
            // the CTA whose slot holds the j-th contribution
            auto contributor = [&](int j) {
                if (split) return (int)blockIdx.x - unit.split_r + (j < unit.split_r ? j : j + 1);
                return (int)blockIdx.x + 1 + j;
            };

            if (unit.kind == kContribution || split) {
                // partial sums that another CTA finishes: to this CTA's slot as they are, then the flag
#pragma unroll 1
                for (int jb = 0; jb < n_jobs_tile; ++jb) {
                    if (split && jb % job_stride == job_start) continue; // (finished here: stays in tensor memory)
                    const int half = jb / kPairs;
                    const uint32_t acc_col = (uint32_t)((buf * MT + half) * BN);
#pragma unroll 1
                    for (int c = (jb % kPairs) * (int)kFetchChunks; c < (jb % kPairs + 1) * (int)kFetchChunks; ++c) {
                        uint32_t v[32];
                        tmem_ld_32x32(tmem_base + ((uint32_t)(32 * q) << 16) + acc_col + (uint32_t)(c * 32), v);
                        tmem_ld_wait();
                        uint8_t *dst = slot_chunk((int)blockIdx.x, half, c);
#pragma unroll
                        for (int pc = 0; pc < 8; ++pc)
                            *reinterpret_cast<uint4 *>(dst + slot_piece(lane, pc)) =
                                make_uint4(v[4 * pc], v[4 * pc + 1], v[4 * pc + 2], v[4 * pc + 3]);
                    }
                }
                tc_fence_before_sync();
                __threadfence(); // this thread's stores are visible to the whole GPU before the flag can be
                __syncwarp();
                if (lane == 0) {
                    if (!split) mbar_arrive(smem_u32(&bars->acc_empty[buf]));
                    mbar_arrive(smem_u32(&bars->epilogue_met));
                }
                // the four epilogue warps meet (a contribution is the CTA's first unit, a split tile its only one: phase 0
                // of this barrier), then one thread raises the flag
                if (!mbar_wait_bounded(smem_u32(&bars->epilogue_met), 0, abort_flag, hooks.limit_us)) break;
                if (warp == 2 && lane == 0) st_release_gpu(sc.flags + blockIdx.x, 1u);
                if (!split) continue;
            }

            // The jobs this CTA finishes.  The parts of other CTAs are in their slots once their flags are up.  They are
            // fetched piece by piece (the kFetchChunks chunks of one job of one contribution) into this warp's buffers,
            // in the order in which they are added: job, contribution.
            const int n_mine = job_start < n_jobs_tile ? (n_jobs_tile - job_start + job_stride - 1) / job_stride : 0;
            const int n_fetches = n_contrib * n_mine;
            uint8_t *fetch_base = smem + q * (kFetchBufs * kFetchBytes);
            int issued = 0, taken = 0;
            auto issue_fetches = [&]() { // lane 0 only
                while (issued < n_fetches && issued - taken < kFetchBufs) {
                    const int j = issued % n_contrib, jb = job_start + (issued / n_contrib) * job_stride;
                    const int b = issued % kFetchBufs;
                    const uint32_t bar = smem_u32(&bars->fetched[q][b]);
                    mbar_arrive_expect_tx(bar, kFetchBytes);
                    bulk_copy_g2s(smem_u32(fetch_base + b * kFetchBytes),
                                  slot_chunk(contributor(j), jb / kPairs, (jb % kPairs) * (int)kFetchChunks), kFetchBytes, bar);
                    ++issued;
                }
            };
            if (n_fetches > 0) {
                bool ok = true;
                for (int j = 0; j < n_contrib && ok; ++j) ok = flag_wait_bounded(sc.flags + contributor(j), abort_flag, hooks.limit_us);
                if (!ok) break;
                fence_proxy_async_smem(); // (the buffers were last touched through the generic proxy or by the tensor core)
                __syncwarp();
                if (lane == 0) issue_fetches();
            }
            bool alive = true;
#pragma unroll 1
            for (int mj = 0; mj < n_mine && alive; ++mj) {
                const int jb = job_start + mj * job_stride;
                const int half = jb / kPairs, c0 = (jb % kPairs) * (int)kFetchChunks;
                const uint32_t acc_col = (uint32_t)((buf * MT + half) * BN);
                const int t = token_of_lane(half);
                int rowsum;
                float scale;
                token_terms(p, gamma, t, rowsum, scale);
                uint32_t v[kFetchChunks][32];
#pragma unroll
                for (int cc = 0; cc < (int)kFetchChunks; ++cc)
                    tmem_ld_32x32(tmem_base + ((uint32_t)(32 * q) << 16) + acc_col + (uint32_t)((c0 + cc) * 32), v[cc]);
                tmem_ld_wait();
                for (int j = 0; j < n_contrib; ++j) {
                    const int b = taken % kFetchBufs;
                    if (!mbar_wait_bounded(smem_u32(&bars->fetched[q][b]), (uint32_t)(taken / kFetchBufs) & 1u, abort_flag,
                                           hooks.limit_us)) {
                        alive = false;
                        break;
                    }
                    const uint8_t *src = fetch_base + b * kFetchBytes;
#pragma unroll
                    for (int cc = 0; cc < (int)kFetchChunks; ++cc) {
#pragma unroll
                        for (int pc = 0; pc < 8; ++pc) {
                            const uint4 w = *reinterpret_cast<const uint4 *>(src + cc * 4096 + slot_piece(lane, pc));
                            v[cc][4 * pc] += w.x;
                            v[cc][4 * pc + 1] += w.y;
                            v[cc][4 * pc + 2] += w.z;
                            v[cc][4 * pc + 3] += w.w;
                        }
                    }
                    __syncwarp(); // every lane has read the buffer before lane 0 refills it
                    ++taken;
                    if (lane == 0) issue_fetches();
                }
                if (!alive) break;
#pragma unroll
                for (int cc = 0; cc < (int)kFetchChunks; ++cc) emit_chunk(p, n0, v[cc], c0 + cc, t, rowsum, scale);
            }
            if (!alive) break;
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bars->acc_empty[buf]));
        }
    }

    // common tail: every thread arrives here, also after an expired wait.  The flag is looked at AFTER the barrier:
    // a thread whose role ended early (the producer of a short matmul, the idle lanes of the one-thread roles) gets
    // here long before a wait of another role can expire.
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) { // (the same for every thread now)
        if (threadIdx.x == 0) atomicExch(status, (int32_t)BITLINEAR_ERR_TIMEOUT);
        // give copies and MMAs that may still be in flight time to land before shared memory and TMEM go away
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == kMmaWarp) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ---- host side ---------------------------------------------------------------------------------

// Tensor maps and parameters of one matmul, for `mt` token tiles per CTA tile.
static cudaError_t fill_problem(GemmProblem &g, const void *packed, const float *gamma, const int8_t *Xq, const float *beta,
                                const int32_t *rowsum, int64_t M, int64_t x_rows, int64_t K, int64_t N, void *out,
                                int out_i32, float qb, int mt, int a_rows, int tile_begin, long long kb_begin, int32_t *status)
{
    if (!encode_tiled_fn()) return cudaErrorNotSupported;
    if (x_rows < M) return cudaErrorInvalidValue;
    // activations: box of a_rows rows; weights: box of 4 row blocks x 2 column tiles
    // (up to 64 tokens: the weight-stationary form reads the weights through the swizzled map)
    if (!encode_activation_map(&g.tmap_x, Xq, x_rows, K, a_rows) ||
        !(a_rows == 64 ? encode_packed_weight_map_swizzled(&g.tmap_w, packed, N, K, BN / kTileRows)
                       : encode_packed_weight_map(&g.tmap_w, packed, N, K, BN / kTileRows)))
        return cudaErrorInvalidValue;
    Params &p = g.p;
    p.gamma = gamma;
    p.beta = beta;
    p.rowsum = rowsum;
    p.out = out;
    p.M = (int)M;
    p.N = (int)N;
    p.KB = (int)((K + BK - 1) / BK);
    p.tiles_m = (int)((M + mt * BM - 1) / (mt * BM));
    p.tiles_n = (int)((N + BN - 1) / BN);
    p.out_i32 = out_i32;
    p.out_32b_aligned = (reinterpret_cast<uintptr_t>(out) % 32 == 0) ? 1 : 0; // (N is a multiple of 16)
    p.tile_begin = tile_begin;
    p.kb_begin = kb_begin;
    p.qb = qb;
    p.status = status;
    return cudaSuccess;
}

// Whether a launch over n_tiles CTA tiles with total_kb k blocks in all deals k-block shares instead of whole tiles.
// Shares cost every CTA one contribution (a pass over its accumulators into its slot, about 5 us) and one wait at the
// end, so they are chosen only where whole tiles would leave a good part of the last round idle: the idle k blocks of
// that round, spread over all SMs, must come to at least kMinIdleKb (about 8 us) per SM, and a share must have at
// least kMinShareKb k blocks.
constexpr long long kMinIdleKb = 12, kMinShareKb = 16, kMaxShareRounds = 6;
static bool deals_shares(long long n_tiles, long long total_kb, int sms)
{
#ifdef BITLINEAR_TUNING // measurement aid, not compiled into the library as build.py builds it
    static const int enabled = [] {
        const char *v = std::getenv("BITLINEAR_PREFILL_SPLIT");
        return (v && *v) ? std::atoi(v) : 1;
    }();
    if (!enabled) return false;
#endif
    if (n_tiles <= 0 || total_kb < kMinShareKb * sms) return false;
    // Only launches of a few rounds: with many rounds the idle part of the last one is a small share of the whole, and
    // whole tiles dealt round-robin keep neighbouring CTAs on neighbouring tiles of one matmul (measured: the 70B-shaped
    // step at 176 tokens, 177 rounds, took 15.0 ms with shares against 11.9 ms with whole tiles).
    if (n_tiles > kMaxShareRounds * sms) return false;
    const long long r = n_tiles % sms;
    if (r == 0) return false;
    const long long idle_kb = (sms - r) * (total_kb / n_tiles) / sms;
    return idle_kb >= kMinIdleKb;
}

// Split tiles.  A launch with so few CTA tiles that at least half of the SMs would have none gives every tile to s CTAs,
// each with 1/s of the tile's k blocks and, afterwards, 1/s of its outputs to finish: every CTA writes the partial sums of
// the jobs it does not finish to its slot, raises its flag, waits for the flags of the other CTAs of its tile and adds
// their parts of its own jobs.  All CTAs are resident at once (grid = n_tiles * s <= SMs, one CTA per SM) and every CTA
// raises its flag before it waits, so the waits end.  s is the largest number with n_tiles * s <= SMs that leaves every
// CTA kMinSplitKb k blocks of the shortest matmul (and at most kMaxSplit: what a CTA writes and fetches grows with s).
constexpr long long kMinSplitKb = 8, kMaxSplit = 8;
static int split_factor(long long n_tiles, long long min_kb, int sms)
{
#ifdef BITLINEAR_TUNING // measurement aid, not compiled into the library as build.py builds it
    static const int enabled = [] {
        const char *v = std::getenv("BITLINEAR_PREFILL_SPLIT_TILES");
        return (v && *v) ? std::atoi(v) : 1;
    }();
    if (!enabled) return 1;
#endif
    if (n_tiles <= 0) return 1;
    long long s = sms / n_tiles;
    if (s > min_kb / kMinSplitKb) s = min_kb / kMinSplitKb;
    if (s > kMaxSplit) s = kMaxSplit;
    return s >= 2 ? (int)s : 1;
}

// Launches the kernel over `n_tiles` CTA tiles: of `one`, or of the `n` matmuls of a device table.
static cudaError_t launch_gemm(const GemmProblem &one, const GemmProblem *table, int n, int n_tiles, long long total_kb,
                               long long min_kb, int mt, int a_rows, int max_M, void *scratch, cudaStream_t stream)
{
    const void *kernel = table ? (mt == 2 ? (const void *)prefill_gemm_kernel<2, true> : (const void *)prefill_gemm_kernel<1, true>)
                               : (mt == 2 ? (const void *)prefill_gemm_kernel<2, false> : (const void *)prefill_gemm_kernel<1, false>);
    int n_stages = stages_that_fit(mt, a_rows);
    const uint32_t smem_bytes = smem_bytes_for(mt, a_rows, n_stages);
    static bool attr_set[64] = {false};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        const void *all[4] = {(const void *)prefill_gemm_kernel<1, false>, (const void *)prefill_gemm_kernel<1, true>,
                              (const void *)prefill_gemm_kernel<2, false>, (const void *)prefill_gemm_kernel<2, true>};
        for (const void *k : all) {
            cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit);
            if (e != cudaSuccess) return e;
        }
        attr_set[dev] = true;
    }
    if (n_tiles <= 0) return cudaSuccess;
    if (a_rows == 64) return launch_decode_tc(one, table, n, n_tiles, max_M, stream); // 17 to 64 tokens: decode_tc.cu
    const int sms = sm_count();
    Schedule sc;
    sc.split = scratch ? split_factor(n_tiles, min_kb, sms) : 1;
    sc.stream_k = sc.split > 1 ? 2 : ((scratch && deals_shares(n_tiles, total_kb, sms)) ? 1 : 0);
    sc.n_tiles = n_tiles;
    sc.total_kb = total_kb;
    sc.flags = reinterpret_cast<uint32_t *>(scratch);
    sc.slots = reinterpret_cast<int32_t *>(reinterpret_cast<char *>(scratch) + kFlagBytes);
    int grid = sc.stream_k == 2 ? n_tiles * sc.split : (sc.stream_k ? sms : (n_tiles < sms ? n_tiles : sms));
    // programmatic dependent launch: see the head of this file
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
    void *args[] = {(void *)&one, (void *)&table, (void *)&n, (void *)&sc, (void *)&a_rows, (void *)&n_stages, (void *)&hooks};
    return cudaLaunchKernelExC(&cfg, kernel, args);
}

} // namespace

int prefill_token_tiles(int64_t max_M) { return max_M > BM ? 2 : 1; }

int64_t prefill_tile_count(int64_t M, int64_t N, int64_t max_M)
{
    const int64_t mt = prefill_token_tiles(max_M);
    return ((M + mt * BM - 1) / (mt * BM)) * ((N + BN - 1) / BN);
}

int64_t prefill_kb_count(int64_t M, int64_t N, int64_t K, int64_t max_M) { return prefill_tile_count(M, N, max_M) * ((K + BK - 1) / BK); }

size_t prefill_scratch_bytes(int64_t n_tiles, int64_t total_kb, int64_t min_kb, int64_t max_M)
{
    static_assert(kFlagBytes >= 4 * 148, "one flag per CTA");
    if (max_M <= 64) return 0; // (the weight-stationary kernel deals whole tiles)
    const int sms = sm_count();
    const int s = split_factor(n_tiles, min_kb, sms);
    if (s < 2 && !deals_shares(n_tiles, total_kb, sms)) return 0;
    const size_t ctas = s >= 2 ? (size_t)n_tiles * (size_t)s : (size_t)sms; // one slot per CTA of the launch
    return kFlagBytes + ctas * (size_t)prefill_token_tiles(max_M) * kSlotTileBytes;
}

size_t prefill_scratch_clear_bytes(int64_t n_tiles, int64_t total_kb, int64_t min_kb, int64_t max_M)
{
    return prefill_scratch_bytes(n_tiles, total_kb, min_kb, max_M) > 0 ? kFlagBytes : 0;
}

// rows of activations per token tile in a TMA stage, for the largest M of a launch
static int prefill_a_rows(int64_t max_M) { return max_M <= 64 ? 64 : BM; }

cudaError_t launch_prefill(const void *packed, const float *gamma, const int8_t *Xq, const float *beta,
                           const int32_t *rowsum, int64_t M, int64_t x_rows, int64_t K, int64_t N, void *out,
                           int out_i32, float qb, WorkspaceHeader *hdr, void *scratch, cudaStream_t stream)
{
    const int mt = prefill_token_tiles(M), a_rows = prefill_a_rows(M);
    GemmProblem g;
    cudaError_t e = fill_problem(g, packed, gamma, Xq, beta, rowsum, M, x_rows, K, N, out, out_i32, qb, mt, a_rows, 0, 0,
                                 &hdr->status);
    if (e != cudaSuccess) return e;
    const int n_tiles = g.p.tiles_m * g.p.tiles_n;
    return launch_gemm(g, nullptr, 1, n_tiles, (long long)n_tiles * g.p.KB, g.p.KB, mt, a_rows, (int)M, scratch, stream);
}

cudaError_t prefill_table_entry(void *slot, const void *packed, const float *gamma, const int8_t *Xq, const float *beta,
                                const int32_t *rowsum, int64_t M, int64_t x_rows, int64_t K, int64_t N, void *out,
                                float qb, int64_t max_M, int tile_begin, int64_t kb_begin, WorkspaceHeader *hdr, int *n_tiles)
{
    GemmProblem g;
    cudaError_t e = fill_problem(g, packed, gamma, Xq, beta, rowsum, M, x_rows, K, N, out, 0, qb, prefill_token_tiles(max_M),
                                 prefill_a_rows(max_M), tile_begin, kb_begin, &hdr->status);
    if (e != cudaSuccess) return e;
    memcpy(slot, &g, sizeof(g));
    *n_tiles = g.p.tiles_m * g.p.tiles_n;
    return cudaSuccess;
}

cudaError_t launch_prefill_table(const void *dev_table, int n, int n_tiles, int64_t total_kb, int64_t min_kb, int64_t max_M,
                                 void *scratch, cudaStream_t stream)
{
    GemmProblem unused{};
    return launch_gemm(unused, reinterpret_cast<const GemmProblem *>(dev_table), n, n_tiles, total_kb, min_kb,
                       prefill_token_tiles(max_M), prefill_a_rows(max_M), (int)max_M, scratch, stream);
}

} // namespace bitlinear
