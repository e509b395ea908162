/*
 * bitlinear.h -- C ABI of the BitLinear forward of BitNet b1.58 on NVIDIA B200 (sm_100a).
 *
 * The library computes, for a weight matrix W [N out, K in] and M tokens X [M, K]:
 *
 *   gamma  = mean_ij |W_ij|                                     (Section 2, Eq. 3)
 *   T_nk   = RoundClip(W_nk / (gamma + eps), -1, 1)             (Section 2, Eq. 1 and Eq. 2)
 *   beta_t = max(max_k |x_tk|, 1e-5)                            (Section 2, per-token absmax, Qb = 127)
 *   q_tk   = clip(round(x_tk * (127 / beta_t)), -127, 127)      (same passage; no zero point)
 *   acc_tn = sum_k q_tk * T_nk           exact, int32           (Section 1: integer additions only)
 *   y_tn   = bf16( float(acc_tn) * ((gamma * beta_t) / 127) )
 *
 * round() is round-half-to-even everywhere; all float steps are single IEEE fp32 operations in the
 * order written, so integer results are reproducible bit for bit.  Ternary weights are stored as
 * 2-bit codes (Section 3, "Memory and Latency": a 2-bit kernel) in the layout described at
 * bitlinear_quantize_weights.
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer owned by the caller unless marked "host".  The library never
 *     allocates or frees device memory.  Inputs are never modified.
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*; NULL = default stream) and
 *     return without synchronising, except bitlinear_poll_status.
 *   - Argument errors are detected on the host, returned at once, and nothing is launched.
 *     Conditions found on the device (a bounded wait that expired) are written to a status word in
 *     the workspace and read back with bitlinear_poll_status.
 *   - Alignment: all device pointers 16-byte aligned; workspaces 256-byte aligned.
 *   - Shapes: N a multiple of 16, K a multiple of 16 with 16 <= K <= 131072 (so |acc| < 2^24 and
 *     float(acc) is exact), 1 <= N <= 2^24, 0 <= M <= 2^20.  M = 0 is a successful no-op, and the
 *     per-token pointers (X, Xq, beta, rowsum, Y, acc) may then be null.
 *   - Only sm_100 devices are supported; other devices give BITLINEAR_ERR_ARCH.  There is no CPU path.
 */
#ifndef BITLINEAR_H_
#define BITLINEAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int bitlinear_status;

enum {
    BITLINEAR_OK = 0,
    BITLINEAR_ERR_ARG = -1,       /* null pointer, negative size, bad enum value */
    BITLINEAR_ERR_SHAPE = -2,     /* N, K or M outside the limits above */
    BITLINEAR_ERR_ALIGN = -3,     /* a pointer is not 16-byte (workspace: 256-byte) aligned */
    BITLINEAR_ERR_WORKSPACE = -4, /* workspace smaller than bitlinear_workspace_bytes says */
    BITLINEAR_ERR_ARCH = -5,      /* current device is not sm_100 */
    BITLINEAR_ERR_CUDA = -6,      /* a CUDA runtime or driver call failed */
    BITLINEAR_ERR_TIMEOUT = -7,   /* a bounded device-side wait expired (device status) */
    BITLINEAR_ERR_RANGE = -8,     /* a weight was non-finite or >= 2^24 in magnitude (reported on the device, as
                                     gamma = NaN; no call returns this code) */
    BITLINEAR_ERR_BADCODE = -9    /* bitlinear_validate_packed found the 2-bit code 3, which no weight has */
};

/* Matmul code paths selectable through the test hook bitlinear_matmul_i32. */
enum {
    BITLINEAR_PATH_AUTO = 0,
    BITLINEAR_PATH_DP4A = 1,   /* scalar dp4a, M <= 8 */
    BITLINEAR_PATH_MMA = 2,    /* warp-level integer MMA on register-unpacked weights, M <= 64 */
    BITLINEAR_PATH_TCGEN05 = 3 /* TMA + tcgen05 int8 tensor cores, any M: up to 64 tokens the weight-stationary kernel, beyond it the GEMM */
};

/* Human-readable name of a status code; never NULL. (host) */
const char *bitlinear_status_string(bitlinear_status s);

/* Bytes of the packed 2-bit weight buffer of an [N, K] matrix: N and K padded to multiples of 64, 4 weights per byte.
 * Returns 0 for shapes the library rejects. (host) */
size_t bitlinear_packed_bytes(int64_t N, int64_t K);

/* Bytes of workspace bitlinear_forward / bitlinear_matmul_i32 need for this shape
 * (int8 activations, beta, row sums, int32 scratch and per-warp lists of the streaming kernel, status word).
 * 0 for rejected shapes. (host) */
size_t bitlinear_workspace_bytes(int64_t M, int64_t N, int64_t K);

/*
 * Weight quantisation and packing: Section 2, Eq. 1-3, plus the 2-bit storage of Section 3.
 *   W       in   fp32 [N, K] row-major (out x in)
 *   eps     in   the epsilon of Eq. 1, added to gamma in the denominator
 *   packed  out  bitlinear_packed_bytes(N, K) bytes
 *   gamma   out  one fp32
 * gamma is the exact sum of |W_ij| (each term truncated to a multiple of 2^-64, accumulated in a
 * 128-bit integer, so the result does not depend on summation order), divided by N*K in double and
 * rounded once to fp32.  If any weight is non-finite or has magnitude >= 2^24, gamma is set to NaN and
 * the packed contents are unspecified.  The first 32 bytes of `packed` serve as scratch while gamma is
 * being computed and are overwritten with their final contents afterwards.
 *
 * Layout.  The code of a weight is T + 1 (0, 1 or 2; 3 never occurs).  The matrix is cut into tiles of
 * 64 rows x 64 columns = 1024 bytes, stored consecutively with the column-tile index fastest; rows N.. and
 * columns K.. up to the next multiple of 64 hold code 1 (weight 0).  One byte holds the codes of four rows at
 * the same column.  Inside a tile, split the row r = n % 64 as 16 f + 8 h + g (f = 0..3, h = 0..1, g = 0..7)
 * and the column c = k % 64 as 16 tq + 8 s + 4 hi + b (tq = 0..3, s = 0..1, hi = 0..1, b = 0..3): the code
 * sits in bits [2 f, 2 f + 1] of byte 512 s + 16 (4 g + tq) + 4 (2 hi + h) + b.  A warp that loads a 512-byte
 * half tile as one 16-byte vector per lane (lane = 4 g + tq) therefore holds, in its four 32-bit words as they
 * are, the A operand of an m16n8k32 integer MMA over rows 8 h + g and columns 16 tq + 8 s + 4 hi + b of all
 * four 16-row groups at once: the operand of group f is w & (0xFF << 2 f & 0xFF, in every byte), i.e. no shift
 * and at most one AND per register (see csrc/decode_gemv.cu), and the tensor-core GEMM expands a tile to
 * bytes with one AND per four weights.
 */
bitlinear_status bitlinear_quantize_weights(const float *W, int64_t N, int64_t K, float eps,
                                            void *packed, float *gamma, void *stream);

/*
 * Activation quantisation: Section 2, paragraph after Eq. 3 (per token, symmetric, [-127, 127]).
 *   X       in   bf16 [M, K] row-major
 *   Xq      out  int8 [M, K]
 *   beta    out  fp32 [M]   clamped absmax of each token
 *   rowsum  out  int32 [M]  sum_k Xq[t, k]  (used by the offset-coded matmul)
 */
bitlinear_status bitlinear_quantize_acts(const void *X, int64_t M, int64_t K,
                                         int8_t *Xq, float *beta, int32_t *rowsum, void *stream);

/*
 * RMSNorm followed by the activation quantiser, in one pass over the token.  Section 2, "LLaMA-alike
 * Components" names RMSNorm among the parts the models are built from and gives no formula; this is the textbook
 * one, x_k = h_k / sqrt(mean_k(h_k^2) + norm_eps) * gain_k, with the arithmetic fixed so that the int8 codes are
 * reproducible bit for bit: the sum of squares is an integer sum, hence order-free, in which every square is cut off
 * (truncated) 30 bits below the unit of the token's largest square -- with E the exponent field of the largest |h_k|,
 * the terms are floor(h_k^2 * 2^(298 - 2E)), which loses less than 2^-44 of the largest square per term --
 * mean = (float)(sum / K) divided in double, r = 1 / sqrt(max(mean + norm_eps, 2^-126)) in IEEE fp32,
 * x_k = (h_k * r) * gain_k, then quantised as above.
 *   H        in   bf16 [M, K] row-major; finite (a token with an infinity or a NaN gets beta = NaN)
 *   gain     in   fp32 [K], 16-byte aligned
 *   norm_eps      >= 0
 *   Xq, beta, rowsum   out, as for bitlinear_quantize_acts
 */
bitlinear_status bitlinear_rmsnorm_quantize_acts(const void *H, const float *gain, float norm_eps, int64_t M, int64_t K,
                                                 int8_t *Xq, float *beta, int32_t *rowsum, void *stream);

/*
 * SwiGLU followed by the activation quantiser, in one pass over the token: what stands in front of the down
 * projection.  Section 2, "LLaMA-alike Components" names SwiGLU and gives no formula; this is the textbook one,
 * h_k = silu(gate_k) * up_k with silu(g) = g / (1 + e^-g), on the bf16 outputs of the gate and up projections, with
 * the arithmetic fixed in fp32 so that the int8 codes are reproducible bit for bit: e^-g by range reduction
 * (n = round(-g * log2 e), r = -g - n * ln 2 with ln 2 in two parts and fused multiply-adds), the Taylor polynomial of
 * degree 7 in Horner's scheme and an exact scaling by 2^n; sigmoid = 1 / (1 + e^-g) with one addition and one IEEE
 * division (0 below g = -87, 1 above 87); h_k = (gate_k * sigmoid) * up_k; then quantised as above.  The product h
 * is never written to memory.
 *   gate, up  in   bf16 [M, K] row-major, 16-byte aligned; finite, with finite products (a token with an infinity
 *                  or a NaN, or whose h overflows fp32, gets beta = NaN)
 *   Xq, beta, rowsum   out, as for bitlinear_quantize_acts
 */
bitlinear_status bitlinear_swiglu_quantize_acts(const void *gate, const void *up, int64_t M, int64_t K,
                                                int8_t *Xq, float *beta, int32_t *rowsum, void *stream);

/*
 * The BitLinear forward: activation quantisation, ternary x int8 matmul with exact int32 accumulation,
 * dequantisation to bf16 (Section 2; no bias, "removes all biases").
 *   packed, gamma   in   from bitlinear_quantize_weights (gamma stays on the device)
 *   X               in   bf16 [M, K]
 *   Y               out  bf16 [M, N]
 *   workspace       scratch, >= bitlinear_workspace_bytes(M, N, K); contents undefined afterwards.
 *                   Two calls that run concurrently must not share a workspace.
 * M <= 16 runs the weight-streaming decode kernel, 17 <= M <= 64 the weight-stationary tensor-core kernel, larger M the
 * tensor-core GEMM.
 */
bitlinear_status bitlinear_forward(const void *packed, const float *gamma, const void *X,
                                   int64_t M, int64_t K, int64_t N, void *Y,
                                   void *workspace, size_t workspace_bytes, void *stream);

/*
 * The same forward with the RMSNorm of bitlinear_rmsnorm_quantize_acts in front of the activation quantiser (one
 * launch normalises and quantises; the matmul and its epilogue are unchanged): Y = BitLinear(RMSNorm(H)).
 */
bitlinear_status bitlinear_forward_rmsnorm(const void *packed, const float *gamma, const void *H, const float *gain,
                                           float norm_eps, int64_t M, int64_t K, int64_t N, void *Y,
                                           void *workspace, size_t workspace_bytes, void *stream);

/*
 * The same forward with the SwiGLU of bitlinear_swiglu_quantize_acts in front of the activation quantiser (one
 * launch forms silu(gate) * up and quantises it; the matmul and its epilogue are unchanged):
 * Y = BitLinear(silu(gate) * up), the down projection of a feed-forward block.  gate, up: bf16 [M, K].
 */
bitlinear_status bitlinear_forward_swiglu(const void *packed, const float *gamma, const void *gate, const void *up,
                                          int64_t M, int64_t K, int64_t N, void *Y,
                                          void *workspace, size_t workspace_bytes, void *stream);

/*
 * The same quantiser and the same forward with activations of fewer bits.  The paper's outlook (Section 4, on long
 * sequences) expects activations to go from 8 bits to 4 bits or fewer; here Q_b = 2^(act_bits - 1) - 1 (7 for 4 bits,
 * 127 for 8) replaces the 127 of Section 2 in the quantiser (s = Q_b / beta, clip to [-Q_b, Q_b]) and in the
 * dequantisation ((gamma * beta_t) / Q_b); everything else, the kernels included, is the forward above.  The codes
 * are still delivered one per byte (Xq int8 [M, K]): this variant changes the arithmetic, not the storage.
 *   act_bits   2 .. 8 (else BITLINEAR_ERR_ARG); 8 gives bitlinear_quantize_acts / bitlinear_forward exactly
 */
bitlinear_status bitlinear_quantize_acts_bits(const void *X, int64_t M, int64_t K, int act_bits,
                                              int8_t *Xq, float *beta, int32_t *rowsum, void *stream);
bitlinear_status bitlinear_forward_act_bits(const void *packed, const float *gamma, const void *X,
                                            int64_t M, int64_t K, int64_t N, int act_bits, void *Y,
                                            void *workspace, size_t workspace_bytes, void *stream);

/*
 * A second storage format: five weights per byte (1.6 bits per weight).  A ternary weight carries log2 3 = 1.58 bits
 * (the paper's title, Section 1), and Section 3 ("Memory and Latency") notes that the 2-bit kernel leaves room: this
 * format moves 4/5 of the bytes and pays for it with a table look-up per stored byte.  The codes c = T + 1 of five rows at
 * one column share a byte as the base-3 number c0 + 3 c1 + 9 c2 + 27 c3 + 81 c4 (0..242).  Tiles are 80 rows x 64 columns
 * = 1024 bytes, stored like the 2-bit tiles (column-tile index fastest; padding rows and columns hold code 1, a padding
 * byte is 121); with r = n % 80 = 16 f + 8 h + g (f = 0..4) and c = k % 64 = 16 tq + 8 s + 4 hi + b, the weight is digit f
 * of byte 512 s + 16 (4 g + tq) + 4 (2 hi + h) + b: the byte positions of the 2-bit format, five rows 16 apart per byte.
 * Eq. 1-3, gamma and every result are those of the 2-bit path bit for bit; only the stored bytes differ.
 *   bitlinear_packed_bytes_trits     bytes of the buffer: ceil(N / 80) * ceil(K / 64) * 1024 (0 for rejected shapes)
 *   bitlinear_quantize_weights_trits as bitlinear_quantize_weights, writing this format
 *   bitlinear_forward_trits          as bitlinear_forward on such a buffer, for M <= 8 tokens (the weight-streaming kernel;
 *                                    more tokens give BITLINEAR_ERR_SHAPE: with many tokens the weights' bytes no longer
 *                                    bound the time, and the 2-bit format is the one to use)
 *   bitlinear_sequence_create_trits  as bitlinear_sequence_create for entries whose weights are all in this format and
 *                                    whose M are all <= 8; run and destroyed like any sequence
 */
size_t bitlinear_packed_bytes_trits(int64_t N, int64_t K);
bitlinear_status bitlinear_quantize_weights_trits(const float *W, int64_t N, int64_t K, float eps,
                                                  void *packed, float *gamma, void *stream);
bitlinear_status bitlinear_forward_trits(const void *packed, const float *gamma, const void *X,
                                         int64_t M, int64_t K, int64_t N, void *Y,
                                         void *workspace, size_t workspace_bytes, void *stream);

/*
 * The same forward for callers that cannot give it a workspace.  (The paper has no counterpart: this is a
 * convenience of the library.)  Some code that wants to run a BitLinear layer is not allowed to allocate
 * device memory at the point of the call -- a plug-in that runs inside another framework's memory pool, a
 * real-time loop that must not touch the allocator, code that runs after the process has been told to
 * stop allocating -- and so has no workspace to hand over.  This entry point calls no allocator of any
 * kind; it uses BITLINEAR_STATIC_WORKSPACE_BYTES of scratch that are part of the library itself (each GPU
 * that loads the library holds them until the process exits).  Inputs and outputs are still the caller's.
 *   - Shapes whose bitlinear_workspace_bytes(M, N, K) exceeds BITLINEAR_STATIC_WORKSPACE_BYTES are refused
 *     with BITLINEAR_ERR_WORKSPACE and nothing is launched.
 *   - The first call on a device looks up the scratch's device address (no allocation, no device work);
 *     make that first call before any stream capture begins on that device.
 *   - All calls on a device share the one scratch area, which still holds what the previous call left:
 *     each call clears what it needs to start at zero, but two calls that overlap on the GPU (different
 *     streams, or the same stream of two host threads without ordering) corrupt each other.  Order them.
 *   - A bounded device-side wait that expires ends the kernel as in bitlinear_forward, but the status word
 *     lies in the library's scratch and cannot be polled through this interface.
 */
#define BITLINEAR_STATIC_WORKSPACE_BYTES ((size_t)8 << 20)
bitlinear_status bitlinear_forward_static(const void *packed, const float *gamma, const void *X,
                                          int64_t M, int64_t K, int64_t N, void *Y, void *stream);

/*
 * A list of independent BitLinear forwards executed by one persistent launch (the seven projections of
 * every decoder layer of a decode step, Section 2 "LLaMA-alike Components").  All inputs X must be
 * ready when the call is enqueued: entries do not depend on each other.  The entries may have different M;
 * the largest decides the kernel for all of them: up to 16 tokens the weight-streaming kernel, from 17 on a
 * tensor-core kernel (weights stationary in tensor memory up to 64 tokens, the GEMM beyond) walking the CTA tiles
 * of all matmuls in one launch.
 */
typedef struct {
    const void *packed; /* device */
    const float *gamma; /* device */
    const void *X;      /* device, bf16 [M, K] */
    void *Y;            /* device, bf16 [M, N] */
    int64_t M, K, N;
} bitlinear_layer_desc;

/* Workspace bytes for a sequence (host array of n descriptors). 0 on invalid input. (host) */
size_t bitlinear_sequence_workspace_bytes(const bitlinear_layer_desc *layers, int n);

/*
 * Builds the launch plan of a sequence: validates the n descriptors (`layers` is a HOST array, free to
 * reuse afterwards), lays the workspace out and copies the descriptor table into it with a synchronous
 * copy.  *out receives an opaque host object; the workspace must stay untouched by the caller until
 * bitlinear_sequence_destroy.  The X and Y pointers are fixed at creation (static decode buffers).
 */
typedef struct bitlinear_sequence bitlinear_sequence;
bitlinear_status bitlinear_sequence_create(const bitlinear_layer_desc *layers, int n, void *workspace,
                                           size_t workspace_bytes, bitlinear_sequence **out);

/*
 * The same with an RMSNorm (see bitlinear_rmsnorm_quantize_acts) in front of the quantiser of chosen entries:
 * `gains` is a HOST array of n DEVICE pointers, gains[i] = the fp32 gain vector [K_i] of entry i (16-byte aligned) or
 * NULL for an entry that is quantised as it is; norm_eps >= 0 serves all of them.  Workspace as for
 * bitlinear_sequence_create.
 */
bitlinear_status bitlinear_sequence_create_rmsnorm(const bitlinear_layer_desc *layers, const float *const *gains,
                                                   float norm_eps, int n, void *workspace, size_t workspace_bytes,
                                                   bitlinear_sequence **out);

/*
 * The same with, besides, a SwiGLU (see bitlinear_swiglu_quantize_acts) in front of the quantiser of chosen entries:
 * `ups` is a HOST array of n DEVICE pointers, ups[i] = the bf16 up input [M_i, K_i] of entry i (16-byte aligned), whose
 * X then is the gate, or NULL for an entry without SwiGLU.  `gains` as above, or NULL when no entry is normalised; an
 * entry takes at most one of the two (else BITLINEAR_ERR_ARG).
 */
bitlinear_status bitlinear_sequence_create_swiglu(const bitlinear_layer_desc *layers, const float *const *gains,
                                                  const void *const *ups, float norm_eps, int n, void *workspace,
                                                  size_t workspace_bytes, bitlinear_sequence **out);

/* The same for weights in the base-3 format (see bitlinear_quantize_weights_trits); every M at most 8. */
bitlinear_status bitlinear_sequence_create_trits(const bitlinear_layer_desc *layers, int n, void *workspace,
                                                 size_t workspace_bytes, bitlinear_sequence **out);

/* Enqueues the whole sequence on `stream`: one batched activation-quantiser launch, one persistent matmul
 * launch that starts while the quantiser is still running (programmatic dependent launch) and one very small
 * finishing launch.  Calls on the same sequence must be stream-ordered, not concurrent.  Once a sequence has run once
 * on the device (the first run sets kernel attributes), later calls may be captured into a CUDA graph. */
bitlinear_status bitlinear_forward_sequence(const bitlinear_sequence *seq, void *stream);

/* The same in two halves, so that a caller can put its own events between them:
 * stage 1 = activation quantiser only (Section 2, per-token absmax), stage 2 = matmul + dequantisation
 * only (needs stage 1 to have run on the same stream first), stage 0 = both. */
bitlinear_status bitlinear_forward_sequence_stage(const bitlinear_sequence *seq, int stage, void *stream);

/* Frees the host object (no device work, no device memory involved).  NULL is allowed. */
void bitlinear_sequence_destroy(bitlinear_sequence *seq);

/*
 * Test hooks.
 * bitlinear_matmul_i32: acc[t, n] = sum_k Xq[t, k] * T[n, k] as int32 [M, N] through the chosen path
 * (the integer matmul of Section 1 in isolation).  Xq int8 [M, K] with values in [-127, 127].
 * bitlinear_unpack_weights: T int8 [N, K] in {-1, 0, 1} from the packed buffer.
 */
bitlinear_status bitlinear_matmul_i32(const void *packed, const int8_t *Xq, int64_t M, int64_t K, int64_t N,
                                      int32_t *acc, int path, void *workspace, size_t workspace_bytes,
                                      void *stream);
bitlinear_status bitlinear_unpack_weights(const void *packed, int64_t N, int64_t K, int8_t *T, void *stream);
/* The same two hooks for the base-3 format (the matmul on the weight-streaming kernel, M <= 8). */
bitlinear_status bitlinear_matmul_i32_trits(const void *packed, const int8_t *Xq, int64_t M, int64_t K, int64_t N,
                                            int32_t *acc, void *workspace, size_t workspace_bytes, void *stream);
bitlinear_status bitlinear_unpack_weights_trits(const void *packed, int64_t N, int64_t K, int8_t *T, void *stream);

/*
 * Checks a packed weight buffer (Section 3, "Memory and Latency": 2-bit storage; a weight is -1, 0 or 1, so the
 * fourth code never occurs): counts the 2-bit fields that hold 3 into *bad_fields (DEVICE, one int32), synchronises
 * `stream` and returns BITLINEAR_ERR_BADCODE if there are any, BITLINEAR_OK otherwise.  A buffer that passes is safe
 * for every kernel; one that does not (a corrupted or foreign file) would give wrong sums, never a fault.
 */
bitlinear_status bitlinear_validate_packed(const void *packed, int64_t N, int64_t K, int32_t *bad_fields, void *stream);

/*
 * Measurement aid (no counterpart in the paper; Section 3, "Energy" is why the prefill matmul is rated against the
 * int8 tensor throughput): what the int8 tensor cores sustain when nothing but MMAs is issued.  One CTA per SM places
 * one 128 x 128-byte and one 256 x 128-byte operand tile of pseudo-random bytes in shared memory once and issues
 * iters x 4 tcgen05.mma kind::i8 of 128 x 256 x 32 on them (1 <= iters <= 2^20; about 0.27 us per iteration).  The
 * caller times the launch; *int_ops (HOST) receives the integer operations it performs, 2 per multiply-add.
 * *status (DEVICE, one int32, set it to 0 first) receives BITLINEAR_ERR_TIMEOUT if the launch's one bounded wait expires.
 */
bitlinear_status bitlinear_probe_int8_peak(int iters, int32_t *status, int64_t *int_ops, void *stream);

/*
 * Test hook for the bounded waits (no counterpart in the paper).  Every device-side wait of the matmul kernels gives
 * up after a limit (2 s), sets the workspace's status word to BITLINEAR_ERR_TIMEOUT and lets the kernel return.  This
 * call arms the NEXT matmul launch of the process (one launch only; the quantiser launch in front of it does not
 * count): its waits give up after limit_us microseconds (0: the default), and, if skip_arrive is non-zero, one
 * producer thread of its first CTA leaves out one barrier arrival (and the copy it announces), so that a wait really
 * runs out.  The launch then
 * ends with BITLINEAR_ERR_TIMEOUT in the status word and unspecified outputs; the workspace is usable again at once.
 * Nothing faults or hangs.  (host)
 */
void bitlinear_test_expire_next_wait(uint32_t limit_us, int skip_arrive);

/* Synchronises `stream`, then copies the workspace's status word to *device_status (host pointer):
 * BITLINEAR_OK or BITLINEAR_ERR_TIMEOUT.  The return value reports the success of the read itself. */
bitlinear_status bitlinear_poll_status(const void *workspace, void *stream, int *device_status);

#ifdef __cplusplus
}
#endif
#endif /* BITLINEAR_H_ */
