// Internal declarations shared by the translation units of the BitLinear CUDA library.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "../../include/bitlinear.h"

namespace bitlinear {

constexpr int kQb = 127;            // Section 2: activations scaled to [-Qb, Qb]
constexpr float kBetaFloor = 1e-5f; // zero-token guard on the per-token absmax
constexpr int kTileRows = 64;       // packed tile: 64 rows x 64 columns = 1024 bytes
constexpr int kTileCols = 64;
constexpr int kTileBytes = 1024;
constexpr int kMaxDecodeM = 64;
// A TMA tensor map over fewer than 32 rows of activations loads markedly slower on B200 (81 against 59 us for the
// same GEMM), so the workspace keeps at least this many rows behind the quantised activations.
constexpr int kMinGemmRows = 32;

// Workspace header (start of every workspace).
struct WorkspaceHeader {
    int32_t status;       // BITLINEAR_OK or BITLINEAR_ERR_TIMEOUT, written by kernels
    uint32_t reserved0[31];
    uint32_t piece_counter; // next dynamically dealt piece of the decode kernel (a 128-byte line of its own)
    uint32_t reserved1[31];
};
static_assert(sizeof(WorkspaceHeader) == 256, "header layout");

// Row blocks a warp of the decode kernel leaves to the finishing launch: (entry index, row block) pairs.
constexpr int kMaxOwned = 15;
constexpr int kMaxDecodeWarps = 2560;
struct OwnedList {
    uint32_t n;
    uint32_t pad;
    uint2 item[kMaxOwned];
};
static_assert(sizeof(OwnedList) == 128, "one line per warp");
constexpr size_t kOwnedListsBytes = sizeof(OwnedList) * kMaxDecodeWarps;

// One matmul of a decode launch, as the kernels see it (device memory or kernel parameter).
struct DecodeEntry {
    const uint4 *packed;   // 2-bit weights
    const float *gamma;    // 1 fp32 (unused when out_i32)
    const __nv_bfloat16 *X; // bf16 [M, K] (input of the quantiser; null for the matmul hook)
    int8_t *Xq;            // int8 activations: [M, K] row-major, or, if xq_tiled, [KB column tiles][M][64 bytes]
    float *beta;           // [M]
    int32_t *rowsum;       // [M]
    void *out;             // bf16 [M, N], or int32 [M, N] when out_i32
    int32_t *acc32;        // scratch [M, N] for row blocks shared by several warps (zero before and after a launch)
    int M, N, K;
    int KB, NB;            // column tiles = ceil(K / 64), row blocks = ceil(N / 64) (base-3 format: ceil(N / 80))
    uint32_t tile_begin;   // index of this entry's first work item in the launch-wide sequence: tiles (NB * KB per
                           // entry) for up to 8 tokens, group tiles (ceil(NB / 8) * KB per entry) beyond: see below
    int token_begin;       // first token of this entry in the batched quantiser's grid
    int out_i32;           // 1: write raw int32 accumulators instead of bf16
    int xq_tiled;          // layout of Xq (the streaming kernel reads tiles, the tensor-core GEMM rows)
    const float *gain;     // null, or [K] fp32: X is normalised first (RMSNorm with this gain) and then quantised
    float norm_eps;        // the RMSNorm's epsilon (added to the mean square)
    float qb;              // largest activation code: 127 (Section 2), or 2^(b-1) - 1 for b-bit activations
    const __nv_bfloat16 *up; // null, or bf16 [M, K]: the quantiser's input is silu(X) * up (SwiGLU; X holds the gate)
};

constexpr int kInlineEntries = 4;
struct InlineTable {
    DecodeEntry e[kInlineEntries];
};

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---- kernel launchers (host side, each defined next to its kernel) ----

// trits: the base-3 format (five weights per byte, tiles of 80 rows) instead of 2-bit codes
cudaError_t launch_absmean_and_pack(const float *W, int64_t N, int64_t K, float eps, void *packed, float *gamma,
                                    cudaStream_t stream, bool trits = false);
cudaError_t launch_unpack(const void *packed, int64_t N, int64_t K, int8_t *T, cudaStream_t stream, bool trits = false);
// *bad (device) = number of 2-bit fields among the `bytes` bytes of a packed buffer that hold the unused code 3.
cudaError_t launch_count_bad_codes(const void *packed, size_t bytes, int32_t *bad, cudaStream_t stream);
// Copies row-major int8 activations [M, K] into the tiled layout [KB][M][64] (columns >= K become 0).
cudaError_t launch_retile_acts(const int8_t *Xq, int64_t M, int64_t K, int8_t *tiled, cudaStream_t stream);

// Quantises the tokens of every entry (entries with X == nullptr are skipped) and zeroes
// `zero_bytes` bytes at `zero_ptr` (control words and split-K scratch) in the same launch.  fronts: bit 0, some
// entry carries a gain vector (RMSNorm in front of the quantiser); bit 1, some entry a second input (SwiGLU).  max_K: the longest token among the entries.
cudaError_t launch_quantize_acts(const InlineTable &inl, const DecodeEntry *table, int n_entries, int total_tokens,
                                 void *zero_ptr, size_t zero_bytes, int fronts, int max_K, cudaStream_t stream);

// The weight-streaming matmul has two kernels: up to 16 tokens every warp streams tiles on its own (one 8-token tile
// per MMA up to 8 tokens, two beyond); from 17 tokens (test hook only) the eight warps of a CTA share the activations and
// the CTA walks group tiles (one row block per warp x 1 column tile).  The sequence of work items of a launch is counted
// accordingly, for the largest token count max_M of the launch.
// Which of the two runs a launch whose largest token count is max_M and whose matmuls have plain_tiles tiles of 64 x 64
// weights (= KiB of packed weights) in all.  Beyond 16 tokens only the lockstep kernel exists.  From 13 to 16 tokens the
// independent warps fetch nearly a KiB of activations per KiB of weights each, which caps them near 4.3 TB/s on the
// path from L2 to the SMs, while the lockstep kernel streams 4.6 TB/s once it runs but takes about 25 us longer to get
// going: it wins from about 1.5 GB of weights per launch on (70B-shaped step at 16 tokens: 3.75 against 3.99 ms; 7B-shaped
// sets of 400 MB: 122 against 104 us).
constexpr uint64_t kWideMinTiles = 1500000;
inline bool decode_is_wide(int max_M, uint64_t plain_tiles) { return max_M > 16 || (max_M >= 13 && plain_tiles >= kWideMinTiles); }
constexpr int decode_wide_warps(int max_M) { return max_M <= 16 ? 8 : 8; }
inline uint32_t decode_items(int NB, int KB, bool wide, int max_M)
{
    const int w = decode_wide_warps(max_M);
    return (uint32_t)(wide ? (NB + w - 1) / w : NB) * (uint32_t)KB;
}

// Persistent weight-streaming matmul over the entries (total_tiles = sum of decode_items over the entries, counted for
// the kernel `wide` names: decode_is_wide).
// path: BITLINEAR_PATH_MMA, or BITLINEAR_PATH_DP4A (first entry only).
// `lists` is scratch of kOwnedListsBytes (no need to clear it).
// trits: the entries' weights are in the base-3 format (five per byte, row blocks of 80 rows: NB = ceil(N / 80)); at
// most 8 tokens then.
cudaError_t launch_decode(const InlineTable &inl, const DecodeEntry *table, int n_entries, uint32_t total_tiles,
                          int max_M, int path, WorkspaceHeader *hdr, OwnedList *lists, cudaStream_t stream, bool trits = false,
                          bool wide = false);

// Tensor-core GEMM (tcgen05): out = dequant(Xq x T^T) (by gamma * beta_t / qb) or raw int32.  x_rows >= M rows of K bytes exist behind
// Xq; the rows past M may hold anything (they only reach accumulator rows that are never stored).
// scratch: prefill_scratch_bytes(...) bytes (256-byte aligned) whose first prefill_scratch_clear_bytes(...) bytes are
// ZERO when the launch starts, or null (then the launch deals whole tiles only).
cudaError_t launch_prefill(const void *packed, const float *gamma, const int8_t *Xq, const float *beta,
                           const int32_t *rowsum, int64_t M, int64_t x_rows, int64_t K, int64_t N, void *out,
                           int out_i32, float qb, WorkspaceHeader *hdr, void *scratch, cudaStream_t stream);

// Dealing k-block shares.  When the CTA tiles of a launch would leave a good part of the SMs idle in their last round,
// the kernel gives every CTA an equal share of the k blocks of all tiles instead; shares begin and end inside tiles, and
// partial sums travel through a scratch slot per CTA.  prefill_scratch_bytes: bytes of scratch a launch over n_tiles CTA
// tiles with total_kb k blocks of 128 columns in all needs (0: it deals whole tiles); prefill_scratch_clear_bytes: how
// many bytes at the start of that scratch must be zero when the launch starts.
int64_t prefill_tile_count(int64_t M, int64_t N, int64_t max_M);
int64_t prefill_kb_count(int64_t M, int64_t N, int64_t K, int64_t max_M); // tiles x k blocks of one matmul
// min_kb: the fewest k blocks any matmul of the launch has (a launch of few tiles splits every tile among several CTAs
// along K when all its matmuls are long enough for that).
size_t prefill_scratch_bytes(int64_t n_tiles, int64_t total_kb, int64_t min_kb, int64_t max_M);
size_t prefill_scratch_clear_bytes(int64_t n_tiles, int64_t total_kb, int64_t min_kb, int64_t max_M);

// The same kernel over the matmuls of a sequence in ONE launch.  The host fills a table of kGemmProblemBytes-sized
// entries (tensor maps + parameters) with prefill_table_entry, copies it to device memory (64-byte aligned) once, and
// launches over all the CTA tiles; max_M = the largest M of the sequence, the same for every entry and the launch
// (it fixes the tile shape: prefill_token_tiles(max_M) token tiles of 128 tokens per CTA tile).  tile_begin, kb_begin:
// the CTA tiles and the k blocks (tiles x k blocks each) of the entries in front of this one.
constexpr size_t kGemmProblemBytes = 384;
int prefill_token_tiles(int64_t max_M);
cudaError_t prefill_table_entry(void *slot, const void *packed, const float *gamma, const int8_t *Xq, const float *beta,
                                const int32_t *rowsum, int64_t M, int64_t x_rows, int64_t K, int64_t N, void *out,
                                float qb, int64_t max_M, int tile_begin, int64_t kb_begin, WorkspaceHeader *hdr, int *n_tiles);
cudaError_t launch_prefill_table(const void *dev_table, int n, int n_tiles, int64_t total_kb, int64_t min_kb, int64_t max_M,
                                 void *scratch, cudaStream_t stream);

// What a matmul launch is told about its bounded device-side waits.  limit_us: how long a wait may last (2 s unless
// a test shortened it).  skip_arrive != 0 is a test device: ONE producer thread of the launch (in CTA 0) leaves out ONE
// barrier arrival and the copy that arrival announces, so that the wait behind it runs out and the kernel's way out
// of an expired wait can be checked; everything else is issued as usual.
struct WaitHooks {
    uint32_t limit_us;
    uint32_t skip_arrive;
};
// The hooks for the next matmul launch: the defaults, or what bitlinear_test_expire_next_wait set (used up by this call).
WaitHooks take_wait_hooks();

// Measurement aid: one CTA per SM issues `iters` x 4 tcgen05.mma kind::i8 (128 x 256 x 32) on operands that stay in
// shared memory.  *ctas (host) = CTAs launched; *status (device) receives BITLINEAR_ERR_TIMEOUT if the final wait expires.
cudaError_t launch_int8_issue_probe(int iters, int32_t *status, int *ctas, cudaStream_t stream);

int sm_count();

} // namespace bitlinear
