// C ABI of the BitLinear library: argument validation, workspace layout, dispatch.
// No arithmetic of the method lives here; every step runs in the kernels.
#include <atomic>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "internal.cuh"
#include "ptx.cuh"

namespace bitlinear {

// The wait hooks of the next matmul launch, packed into one word so that setting and taking them are single atomic
// operations: bits 0..30 the limit in microseconds (0: the default), bit 31 the skipped arrival.
static std::atomic<uint32_t> g_next_wait_hooks{0};

WaitHooks take_wait_hooks()
{
    const uint32_t v = g_next_wait_hooks.exchange(0u);
    WaitHooks h;
    h.limit_us = (v & 0x7FFFFFFFu) ? (v & 0x7FFFFFFFu) : ptx::kWaitLimitUs;
    h.skip_arrive = v >> 31;
    return h;
}

int sm_count()
{
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

namespace {

bool device_is_sm100()
{
    static int cached[64] = {0}; // 0 unknown, 1 yes, 2 no
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    if (cached[dev] == 0) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return false;
        cached[dev] = (major == 10) ? 1 : 2;
    }
    return cached[dev] == 1;
}

inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

bitlinear_status check_shape(int64_t M, int64_t N, int64_t K)
{
    if (M < 0 || M > (1 << 20)) return BITLINEAR_ERR_SHAPE;
    if (N < 16 || N > (1 << 24) || (N % 16) != 0) return BITLINEAR_ERR_SHAPE;
    if (K < 16 || K > 131072 || (K % 16) != 0) return BITLINEAR_ERR_SHAPE;
    return BITLINEAR_OK;
}

// Measurement aid, compiled in only with -DBITLINEAR_TUNING (the library as built by build.py reads no environment
// variable).
int env_int(const char *name, int fallback)
{
#ifdef BITLINEAR_TUNING
    const char *v = std::getenv(name);
    if (!v || !*v) return fallback;
    return std::atoi(v);
#else
    (void)name;
    return fallback;
#endif
}

struct Layout {
    size_t acc32, table, lists, xq, beta, rowsum, total;
};

inline int64_t row_blocks(int64_t N) { return (N + kTileRows - 1) / kTileRows; }
inline int64_t col_tiles(int64_t K) { return (K + kTileCols - 1) / kTileCols; }

inline int64_t gemm_k_blocks(int64_t K) { return (K + 127) / 128; }
constexpr int kMaxTritM = 8; // the base-3 format runs on the weight-streaming kernel for up to 8 tokens only
inline int64_t trit_row_blocks(int64_t N) { return (N + 79) / 80; }

// Workspace of one matmul: [header | int32 scratch | per-warp lists | Xq | beta | rowsum].  The scratch serves the
// weight-streaming kernel (sums of row blocks shared by several warps, at most 64 tokens) or the GEMM (flags and a slot
// of partial sums per CTA when it deals k-block shares), whichever is larger, so that the layout does not depend on the kernel chosen.
Layout single_layout(int64_t M, int64_t N, int64_t K)
{
    Layout L{};
    size_t off = sizeof(WorkspaceHeader);
    L.acc32 = off;
    const size_t decode_scratch = (size_t)(M < kMaxDecodeM ? M : kMaxDecodeM) * N * 4;
    const size_t gemm_scratch = M > 0 ? prefill_scratch_bytes(prefill_tile_count(M, N, M), prefill_kb_count(M, N, K, M), gemm_k_blocks(K), M) : 0;
    off += align_up(decode_scratch > gemm_scratch ? decode_scratch : gemm_scratch, 256);
    L.table = off; // end of what is cleared before every call
    L.lists = off;
    off += align_up(kOwnedListsBytes, 256);
    L.xq = off;
    // room for either layout of the int8 activations; at least kMinGemmRows rows (see launch_prefill)
    off += align_up((size_t)(M < kMinGemmRows ? kMinGemmRows : M) * col_tiles(K) * kTileCols, 256);
    L.beta = off;
    off += align_up((size_t)M * 4, 256);
    L.rowsum = off;
    off += align_up((size_t)M * 4, 256);
    L.total = off;
    return L;
}

__global__ void rowsum_kernel(const int8_t *__restrict__ Xq, int K, int32_t *__restrict__ rowsum)
{
    const int t = blockIdx.x;
    int s = 0;
    for (int k = threadIdx.x; k < K; k += blockDim.x) s += Xq[(size_t)t * K + k];
    s = __reduce_add_sync(0xffffffffu, s);
    __shared__ int part[8];
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        int tot = 0;
        for (int w = 0; w < 8; ++w) tot += part[w];
        rowsum[t] = tot;
    }
}

// From 17 tokens on a matmul goes to the tensor cores (the launchers of prefill_gemm.cu pick the weight-stationary kernel
// up to 64 tokens and the GEMM beyond): measured on 110080 x 4096 (whole forward, the 113 MB of weights resident in L2),
// the weight-streaming kernel takes 48 us at 16 tokens, 92 us at 32 and 174 us at 64; the weight-stationary kernel 39, 40
// and 42 us at 17, 32 and 64 tokens, the GEMM 57 us at 128.
// (In a -DBITLINEAR_TUNING build BITLINEAR_TCGEN05_MIN_M moves the switch-over point.)
bool use_tcgen05_for(int64_t M)
{
    static const int min_m = env_int("BITLINEAR_TCGEN05_MIN_M", 17);
    return M > kMaxDecodeM || M >= min_m;
}

// Fills one DecodeEntry for a matmul whose workspace part starts at `base`.
void fill_entry(DecodeEntry &e, const void *packed, const float *gamma, const void *X, int64_t M, int64_t K,
                int64_t N, void *out, int out_i32, char *base, const Layout &L, bool trits = false)
{
    e.packed = reinterpret_cast<const uint4 *>(packed);
    e.gamma = gamma;
    e.X = reinterpret_cast<const __nv_bfloat16 *>(X);
    e.Xq = reinterpret_cast<int8_t *>(base + L.xq);
    e.beta = reinterpret_cast<float *>(base + L.beta);
    e.rowsum = reinterpret_cast<int32_t *>(base + L.rowsum);
    e.out = out;
    e.acc32 = reinterpret_cast<int32_t *>(base + L.acc32);
    e.M = (int)M;
    e.N = (int)N;
    e.K = (int)K;
    e.KB = (int)col_tiles(K);
    e.NB = (int)(trits ? trit_row_blocks(N) : row_blocks(N));
    e.tile_begin = 0;
    e.token_begin = 0;
    e.out_i32 = out_i32;
    e.xq_tiled = 0;
    e.gain = nullptr;
    e.norm_eps = 0.0f;
    e.up = nullptr;
    e.qb = (float)kQb;
}

// Runs the matmul + epilogue of one entry whose activations are already quantised.
// x_rows: rows of int8 activations that exist behind e.Xq (>= e.M; the rows past e.M may hold anything).
// split_scratch: the GEMM's scratch with its flags zeroed, or null (then it deals whole tiles only).
bitlinear_status run_matmul(DecodeEntry e, int path, char *ws, size_t lists_offset, int64_t x_rows, void *split_scratch,
                            cudaStream_t stream, bool trits = false)
{
    WorkspaceHeader *hdr = reinterpret_cast<WorkspaceHeader *>(ws);
    OwnedList *lists = reinterpret_cast<OwnedList *>(ws + lists_offset);
    const bool tc = !trits && ((path == BITLINEAR_PATH_TCGEN05) || (path == BITLINEAR_PATH_AUTO && use_tcgen05_for(e.M)));
    if (tc) {
        cudaError_t err = launch_prefill(e.packed, e.gamma, e.Xq, e.beta, e.rowsum, e.M, x_rows, e.K, e.N, e.out, e.out_i32,
                                         e.qb, hdr, split_scratch, stream);
        return err == cudaSuccess ? BITLINEAR_OK : BITLINEAR_ERR_CUDA;
    }
    if (e.M > kMaxDecodeM) return BITLINEAR_ERR_SHAPE; // the weight-streaming kernel takes at most 64 tokens
    InlineTable inl{};
    inl.e[0] = e;
    const bool wide = !trits && decode_is_wide(e.M, (uint64_t)e.NB * (uint64_t)e.KB);
    cudaError_t err = launch_decode(inl, nullptr, 1, decode_items(e.NB, e.KB, wide, e.M), e.M,
                                    path == BITLINEAR_PATH_DP4A ? path : BITLINEAR_PATH_MMA, hdr, lists, stream, trits, wide);
    if (err != cudaSuccess) return BITLINEAR_ERR_CUDA;
    return BITLINEAR_OK;
}

} // namespace
} // namespace bitlinear

using namespace bitlinear;

extern "C" {

const char *bitlinear_status_string(bitlinear_status s)
{
    switch (s) {
    case BITLINEAR_OK: return "ok";
    case BITLINEAR_ERR_ARG: return "invalid argument";
    case BITLINEAR_ERR_SHAPE: return "unsupported shape";
    case BITLINEAR_ERR_ALIGN: return "misaligned pointer";
    case BITLINEAR_ERR_WORKSPACE: return "workspace too small";
    case BITLINEAR_ERR_ARCH: return "device is not sm_100";
    case BITLINEAR_ERR_CUDA: return "CUDA call failed";
    case BITLINEAR_ERR_TIMEOUT: return "device-side wait timed out";
    case BITLINEAR_ERR_RANGE: return "weight out of range";
    case BITLINEAR_ERR_BADCODE: return "packed weights hold the unused 2-bit code";
    default: return "unknown status";
    }
}

size_t bitlinear_packed_bytes(int64_t N, int64_t K)
{
    if (check_shape(0, N, K) != BITLINEAR_OK) return 0;
    return (size_t)(row_blocks(N) * col_tiles(K)) * kTileBytes;
}

size_t bitlinear_packed_bytes_trits(int64_t N, int64_t K)
{
    if (check_shape(0, N, K) != BITLINEAR_OK) return 0;
    return (size_t)(trit_row_blocks(N) * col_tiles(K)) * kTileBytes;
}

size_t bitlinear_workspace_bytes(int64_t M, int64_t N, int64_t K)
{
    if (check_shape(M, N, K) != BITLINEAR_OK) return 0;
    return single_layout(M, N, K).total;
}

namespace {
bitlinear_status quantize_weights_impl(const float *W, int64_t N, int64_t K, float eps, void *packed, float *gamma,
                                       void *stream, bool trits)
{
    if (!W || !packed || !gamma || !(eps >= 0.0f)) return BITLINEAR_ERR_ARG;
    bitlinear_status st = check_shape(0, N, K);
    if (st != BITLINEAR_OK) return st;
    if (!aligned(W, 16) || !aligned(packed, 16) || !aligned(gamma, 4)) return BITLINEAR_ERR_ALIGN;
    if (!device_is_sm100()) return BITLINEAR_ERR_ARCH;
    cudaError_t err = launch_absmean_and_pack(W, N, K, eps, packed, gamma, (cudaStream_t)stream, trits);
    return err == cudaSuccess ? BITLINEAR_OK : BITLINEAR_ERR_CUDA;
}
} // namespace

bitlinear_status bitlinear_quantize_weights(const float *W, int64_t N, int64_t K, float eps, void *packed,
                                            float *gamma, void *stream)
{
    return quantize_weights_impl(W, N, K, eps, packed, gamma, stream, false);
}

bitlinear_status bitlinear_quantize_weights_trits(const float *W, int64_t N, int64_t K, float eps, void *packed,
                                                  float *gamma, void *stream)
{
    return quantize_weights_impl(W, N, K, eps, packed, gamma, stream, true);
}

namespace {
// gain == null and up == null: the plain quantiser; gain: RMSNorm in front; up: SwiGLU in front (X is the gate)
// act_bits: 8 (Section 2), or fewer
bitlinear_status quantize_acts_rows(const void *X, const void *up, const float *gain, float norm_eps, int act_bits,
                                    int64_t M, int64_t K, int8_t *Xq, float *beta, int32_t *rowsum, void *stream)
{
    if (act_bits < 2 || act_bits > 8) return BITLINEAR_ERR_ARG;
    if (M > 0 && (!X || !Xq || !beta || !rowsum)) return BITLINEAR_ERR_ARG;
    bitlinear_status st = check_shape(M, 16, K);
    if (st != BITLINEAR_OK) return st;
    if (!aligned(X, 16) || !aligned(Xq, 16) || !aligned(beta, 4) || !aligned(rowsum, 4)) return BITLINEAR_ERR_ALIGN;
    if (gain && !aligned(gain, 16)) return BITLINEAR_ERR_ALIGN;
    if (up && !aligned(up, 16)) return BITLINEAR_ERR_ALIGN;
    if (!device_is_sm100()) return BITLINEAR_ERR_ARCH;
    if (M == 0) return BITLINEAR_OK;
    InlineTable inl{};
    DecodeEntry &e = inl.e[0];
    e.X = reinterpret_cast<const __nv_bfloat16 *>(X);
    e.Xq = Xq;
    e.beta = beta;
    e.rowsum = rowsum;
    e.M = (int)M;
    e.K = (int)K;
    e.gain = gain;
    e.norm_eps = norm_eps;
    e.up = reinterpret_cast<const __nv_bfloat16 *>(up);
    e.qb = (float)((1 << (act_bits - 1)) - 1);
    cudaError_t err = launch_quantize_acts(inl, nullptr, 1, (int)M, nullptr, 0, (gain ? 1 : 0) | (up ? 2 : 0), (int)K,
                                           (cudaStream_t)stream);
    return err == cudaSuccess ? BITLINEAR_OK : BITLINEAR_ERR_CUDA;
}
} // namespace

bitlinear_status bitlinear_quantize_acts(const void *X, int64_t M, int64_t K, int8_t *Xq, float *beta,
                                         int32_t *rowsum, void *stream)
{
    return quantize_acts_rows(X, nullptr, nullptr, 0.0f, 8, M, K, Xq, beta, rowsum, stream);
}

bitlinear_status bitlinear_quantize_acts_bits(const void *X, int64_t M, int64_t K, int act_bits, int8_t *Xq, float *beta,
                                              int32_t *rowsum, void *stream)
{
    return quantize_acts_rows(X, nullptr, nullptr, 0.0f, act_bits, M, K, Xq, beta, rowsum, stream);
}

bitlinear_status bitlinear_rmsnorm_quantize_acts(const void *H, const float *gain, float norm_eps, int64_t M, int64_t K,
                                                 int8_t *Xq, float *beta, int32_t *rowsum, void *stream)
{
    if (!gain || !(norm_eps >= 0.0f)) return BITLINEAR_ERR_ARG;
    return quantize_acts_rows(H, nullptr, gain, norm_eps, 8, M, K, Xq, beta, rowsum, stream);
}

bitlinear_status bitlinear_swiglu_quantize_acts(const void *gate, const void *up, int64_t M, int64_t K, int8_t *Xq,
                                                float *beta, int32_t *rowsum, void *stream)
{
    if (M > 0 && !up) return BITLINEAR_ERR_ARG;
    return quantize_acts_rows(gate, up, nullptr, 0.0f, 8, M, K, Xq, beta, rowsum, stream);
}

namespace {
bitlinear_status forward_impl(const void *packed, const float *gamma, const void *X, const void *up, const float *gain,
                              float norm_eps, int act_bits, int64_t M, int64_t K, int64_t N, void *Y, void *workspace,
                              size_t workspace_bytes, void *stream, bool trits = false);
}

bitlinear_status bitlinear_forward(const void *packed, const float *gamma, const void *X, int64_t M, int64_t K,
                                   int64_t N, void *Y, void *workspace, size_t workspace_bytes, void *stream)
{
    return forward_impl(packed, gamma, X, nullptr, nullptr, 0.0f, 8, M, K, N, Y, workspace, workspace_bytes, stream);
}

bitlinear_status bitlinear_forward_rmsnorm(const void *packed, const float *gamma, const void *H, const float *gain,
                                           float norm_eps, int64_t M, int64_t K, int64_t N, void *Y, void *workspace,
                                           size_t workspace_bytes, void *stream)
{
    if (!gain || !(norm_eps >= 0.0f)) return BITLINEAR_ERR_ARG;
    if (!aligned(gain, 16)) return BITLINEAR_ERR_ALIGN;
    return forward_impl(packed, gamma, H, nullptr, gain, norm_eps, 8, M, K, N, Y, workspace, workspace_bytes, stream);
}

bitlinear_status bitlinear_forward_swiglu(const void *packed, const float *gamma, const void *gate, const void *up,
                                          int64_t M, int64_t K, int64_t N, void *Y, void *workspace,
                                          size_t workspace_bytes, void *stream)
{
    if (M > 0 && !up) return BITLINEAR_ERR_ARG;
    if (!aligned(up, 16)) return BITLINEAR_ERR_ALIGN;
    return forward_impl(packed, gamma, gate, up, nullptr, 0.0f, 8, M, K, N, Y, workspace, workspace_bytes, stream);
}

bitlinear_status bitlinear_forward_trits(const void *packed, const float *gamma, const void *X, int64_t M, int64_t K,
                                         int64_t N, void *Y, void *workspace, size_t workspace_bytes, void *stream)
{
    return forward_impl(packed, gamma, X, nullptr, nullptr, 0.0f, 8, M, K, N, Y, workspace, workspace_bytes, stream, true);
}

bitlinear_status bitlinear_forward_act_bits(const void *packed, const float *gamma, const void *X, int64_t M, int64_t K,
                                            int64_t N, int act_bits, void *Y, void *workspace, size_t workspace_bytes,
                                            void *stream)
{
    return forward_impl(packed, gamma, X, nullptr, nullptr, 0.0f, act_bits, M, K, N, Y, workspace, workspace_bytes, stream);
}

namespace {
// gain == null: no normalisation in front of the quantiser; up != null: X is the gate of a SwiGLU in front of it
bitlinear_status forward_impl(const void *packed, const float *gamma, const void *X, const void *up, const float *gain,
                              float norm_eps, int act_bits, int64_t M, int64_t K, int64_t N, void *Y, void *workspace,
                              size_t workspace_bytes, void *stream, bool trits)
{
    if (act_bits < 2 || act_bits > 8) return BITLINEAR_ERR_ARG;
    if (trits && M > kMaxTritM) return BITLINEAR_ERR_SHAPE;
    if (!packed || !gamma || !workspace || (M > 0 && (!X || !Y))) return BITLINEAR_ERR_ARG;
    bitlinear_status st = check_shape(M, N, K);
    if (st != BITLINEAR_OK) return st;
    if (!aligned(packed, 16) || !aligned(X, 16) || !aligned(Y, 16) || !aligned(gamma, 4)) return BITLINEAR_ERR_ALIGN;
    if (!aligned(workspace, 256)) return BITLINEAR_ERR_ALIGN;
    const Layout L = single_layout(M, N, K);
    if (workspace_bytes < L.total) return BITLINEAR_ERR_WORKSPACE;
    if (!device_is_sm100()) return BITLINEAR_ERR_ARCH;
    if (M == 0) return BITLINEAR_OK;
    char *ws = reinterpret_cast<char *>(workspace);
    InlineTable inl{};
    fill_entry(inl.e[0], packed, gamma, X, M, K, N, Y, 0, ws, L, trits);
    const bool tc = !trits && use_tcgen05_for(M);
    inl.e[0].xq_tiled = tc ? 0 : 1;
    inl.e[0].gain = gain;
    inl.e[0].norm_eps = norm_eps;
    inl.e[0].up = reinterpret_cast<const __nv_bfloat16 *>(up);
    inl.e[0].qb = (float)((1 << (act_bits - 1)) - 1);
    // quantise the tokens; the same launch clears the header and the scratch of the kernel that follows, if it uses it
    const size_t clear = tc ? prefill_scratch_clear_bytes(prefill_tile_count(M, N, M), prefill_kb_count(M, N, K, M), gemm_k_blocks(K), M) : 0;
    const bool split = clear > 0;
    const size_t zero_bytes = tc ? L.acc32 + align_up(clear, 256) : L.table;
    cudaError_t err = launch_quantize_acts(inl, nullptr, 1, (int)M, ws, zero_bytes, (gain ? 1 : 0) | (up ? 2 : 0), (int)K,
                                           (cudaStream_t)stream);
    if (err != cudaSuccess) return BITLINEAR_ERR_CUDA;
    return run_matmul(inl.e[0], BITLINEAR_PATH_AUTO, ws, L.lists, M < kMinGemmRows ? kMinGemmRows : M,
                      split ? ws + L.acc32 : nullptr, (cudaStream_t)stream, trits);
}
} // namespace

namespace {
bitlinear_status matmul_i32_impl(const void *packed, const int8_t *Xq, int64_t M, int64_t K, int64_t N, int32_t *acc,
                                 int path, void *workspace, size_t workspace_bytes, void *stream, bool trits);
}

bitlinear_status bitlinear_matmul_i32(const void *packed, const int8_t *Xq, int64_t M, int64_t K, int64_t N,
                                      int32_t *acc, int path, void *workspace, size_t workspace_bytes, void *stream)
{
    return matmul_i32_impl(packed, Xq, M, K, N, acc, path, workspace, workspace_bytes, stream, false);
}

bitlinear_status bitlinear_matmul_i32_trits(const void *packed, const int8_t *Xq, int64_t M, int64_t K, int64_t N,
                                            int32_t *acc, void *workspace, size_t workspace_bytes, void *stream)
{
    if (M > kMaxTritM) return BITLINEAR_ERR_SHAPE;
    return matmul_i32_impl(packed, Xq, M, K, N, acc, BITLINEAR_PATH_MMA, workspace, workspace_bytes, stream, true);
}

namespace {
bitlinear_status matmul_i32_impl(const void *packed, const int8_t *Xq, int64_t M, int64_t K, int64_t N, int32_t *acc,
                                 int path, void *workspace, size_t workspace_bytes, void *stream, bool trits)
{
    if (!packed || !workspace || (M > 0 && (!Xq || !acc))) return BITLINEAR_ERR_ARG;
    if (path < BITLINEAR_PATH_AUTO || path > BITLINEAR_PATH_TCGEN05) return BITLINEAR_ERR_ARG;
    bitlinear_status st = check_shape(M, N, K);
    if (st != BITLINEAR_OK) return st;
    if (path == BITLINEAR_PATH_DP4A && M > 8) return BITLINEAR_ERR_SHAPE;
    if (path == BITLINEAR_PATH_MMA && M > kMaxDecodeM) return BITLINEAR_ERR_SHAPE;
    if (!aligned(packed, 16) || !aligned(Xq, 16) || !aligned(acc, 16)) return BITLINEAR_ERR_ALIGN;
    if (!aligned(workspace, 256)) return BITLINEAR_ERR_ALIGN;
    const Layout L = single_layout(M, N, K);
    if (workspace_bytes < L.total) return BITLINEAR_ERR_WORKSPACE;
    if (!device_is_sm100()) return BITLINEAR_ERR_ARCH;
    if (M == 0) return BITLINEAR_OK;
    char *ws = reinterpret_cast<char *>(workspace);
    cudaStream_t s = (cudaStream_t)stream;
    const bool tc = !trits && ((path == BITLINEAR_PATH_TCGEN05) || (path == BITLINEAR_PATH_AUTO && use_tcgen05_for(M)));
    InlineTable inl{};
    fill_entry(inl.e[0], packed, nullptr, nullptr, M, K, N, acc, 1, ws, L, trits);
    const size_t clear = tc ? prefill_scratch_clear_bytes(prefill_tile_count(M, N, M), prefill_kb_count(M, N, K, M), gemm_k_blocks(K), M) : 0;
    const bool split = clear > 0;
    const size_t zero_bytes = tc ? L.acc32 + align_up(clear, 256) : L.table;
    cudaError_t err = launch_quantize_acts(inl, nullptr, 1, 0, ws, zero_bytes, false, (int)K, s);
    if (err != cudaSuccess) return BITLINEAR_ERR_CUDA;
    if (tc) {
        inl.e[0].Xq = const_cast<int8_t *>(Xq); // the GEMM reads the caller's rows in place
    } else {
        inl.e[0].xq_tiled = 1; // the streaming kernels read tiles: copy the rows into the workspace
        if (launch_retile_acts(Xq, M, K, inl.e[0].Xq, s) != cudaSuccess) return BITLINEAR_ERR_CUDA;
    }
    rowsum_kernel<<<(unsigned)M, 256, 0, s>>>(Xq, (int)K, inl.e[0].rowsum);
    if (cudaGetLastError() != cudaSuccess) return BITLINEAR_ERR_CUDA;
    return run_matmul(inl.e[0], path, ws, L.lists, M, split ? ws + L.acc32 : nullptr, s, trits); // (the caller's rows: exactly M)
}
} // namespace

namespace {
bitlinear_status unpack_impl(const void *packed, int64_t N, int64_t K, int8_t *T, void *stream, bool trits)
{
    if (!packed || !T) return BITLINEAR_ERR_ARG;
    bitlinear_status st = check_shape(0, N, K);
    if (st != BITLINEAR_OK) return st;
    if (!aligned(packed, 16)) return BITLINEAR_ERR_ALIGN;
    if (!device_is_sm100()) return BITLINEAR_ERR_ARCH;
    cudaError_t err = launch_unpack(packed, N, K, T, (cudaStream_t)stream, trits);
    return err == cudaSuccess ? BITLINEAR_OK : BITLINEAR_ERR_CUDA;
}
} // namespace

bitlinear_status bitlinear_unpack_weights(const void *packed, int64_t N, int64_t K, int8_t *T, void *stream)
{
    return unpack_impl(packed, N, K, T, stream, false);
}

bitlinear_status bitlinear_unpack_weights_trits(const void *packed, int64_t N, int64_t K, int8_t *T, void *stream)
{
    return unpack_impl(packed, N, K, T, stream, true);
}

bitlinear_status bitlinear_validate_packed(const void *packed, int64_t N, int64_t K, int32_t *bad_fields, void *stream)
{
    if (!packed || !bad_fields) return BITLINEAR_ERR_ARG;
    bitlinear_status st = check_shape(0, N, K);
    if (st != BITLINEAR_OK) return st;
    if (!aligned(packed, 16) || !aligned(bad_fields, 4)) return BITLINEAR_ERR_ALIGN;
    if (!device_is_sm100()) return BITLINEAR_ERR_ARCH;
    cudaStream_t s = (cudaStream_t)stream;
    if (launch_count_bad_codes(packed, bitlinear_packed_bytes(N, K), bad_fields, s) != cudaSuccess) return BITLINEAR_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return BITLINEAR_ERR_CUDA;
    int32_t n = 0;
    if (cudaMemcpy(&n, bad_fields, sizeof n, cudaMemcpyDeviceToHost) != cudaSuccess) return BITLINEAR_ERR_CUDA;
    return n == 0 ? BITLINEAR_OK : BITLINEAR_ERR_BADCODE;
}

bitlinear_status bitlinear_probe_int8_peak(int iters, int32_t *status, int64_t *int_ops, void *stream)
{
    if (!status || !int_ops || iters < 1 || iters > (1 << 20)) return BITLINEAR_ERR_ARG;
    if (!aligned(status, 4)) return BITLINEAR_ERR_ALIGN;
    if (!device_is_sm100()) return BITLINEAR_ERR_ARCH;
    int ctas = 0;
    if (launch_int8_issue_probe(iters, status, &ctas, (cudaStream_t)stream) != cudaSuccess) return BITLINEAR_ERR_CUDA;
    *int_ops = (int64_t)ctas * iters * 4 * (2ll * 128 * 256 * 32);
    return BITLINEAR_OK;
}

void bitlinear_test_expire_next_wait(uint32_t limit_us, int skip_arrive)
{
    if (limit_us > 0x7FFFFFFFu) limit_us = 0x7FFFFFFFu;
    g_next_wait_hooks.store(limit_us | (skip_arrive ? 0x80000000u : 0u));
}

bitlinear_status bitlinear_poll_status(const void *workspace, void *stream, int *device_status)
{
    if (!workspace || !device_status) return BITLINEAR_ERR_ARG;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return BITLINEAR_ERR_CUDA;
    int32_t v = 0;
    if (cudaMemcpy(&v, workspace, sizeof v, cudaMemcpyDeviceToHost) != cudaSuccess) return BITLINEAR_ERR_CUDA;
    *device_status = (int)v;
    return BITLINEAR_OK;
}

// ---- forward without a caller workspace ---------------------------------------------------------
// Scratch for bitlinear_forward_static: part of the library's device image, so every GPU that loads the
// library holds these bytes until the process exits.  In host code this name is only a handle; the
// device address comes from cudaGetSymbolAddress.
constexpr size_t kStaticWorkspaceBytes = BITLINEAR_STATIC_WORKSPACE_BYTES;
static __device__ __align__(256) unsigned char g_static_workspace[kStaticWorkspaceBytes];

bitlinear_status bitlinear_forward_static(const void *packed, const float *gamma, const void *X, int64_t M, int64_t K,
                                          int64_t N, void *Y, void *stream)
{
    bitlinear_status st = check_shape(M, N, K);
    if (st != BITLINEAR_OK) return st;
    if (single_layout(M, N, K).total > kStaticWorkspaceBytes) return BITLINEAR_ERR_WORKSPACE;
    // the checks bitlinear_forward would make, before the device is asked for anything
    if (!packed || !gamma || (M > 0 && (!X || !Y))) return BITLINEAR_ERR_ARG;
    if (!aligned(packed, 16) || !aligned(X, 16) || !aligned(Y, 16) || !aligned(gamma, 4)) return BITLINEAR_ERR_ALIGN;
    if (!device_is_sm100()) return BITLINEAR_ERR_ARCH;
    // device address of the scratch, looked up once per device while that device is current (two host threads that
    // get here together both look it up and store the same value)
    static std::atomic<void *> address[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return BITLINEAR_ERR_CUDA;
    if (!address[dev].load(std::memory_order_acquire)) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_workspace) != cudaSuccess || !p) return BITLINEAR_ERR_CUDA;
        address[dev].store(p, std::memory_order_release);
    }
    // bitlinear_forward clears the part of the workspace that has to start at zero on every call
    return bitlinear_forward(packed, gamma, X, M, K, N, Y, address[dev].load(std::memory_order_acquire),
                             kStaticWorkspaceBytes, stream);
}

// ---- sequences -------------------------------------------------------------------------------
// Workspace: [header | all acc32 | descriptor table | per-warp lists | GEMM table | per-entry Xq, beta, rowsum]
// A sequence whose largest matmul has 17 tokens or more runs all its matmuls in one launch on the tensor cores (up to 64
// tokens the weight-stationary kernel of decode_tc.cu, beyond it the GEMM; no int32 scratch, row-major activations with at
// least kMinGemmRows rows each); otherwise in one launch of the weight-streaming kernel.

struct bitlinear_sequence {
    char *workspace;
    bitlinear::OwnedList *lists;
    int n, tokens, max_M, max_K;
    uint32_t tiles;
    size_t zero_bytes;
    const bitlinear::DecodeEntry *dev_table; // inside the workspace, or null when the table is inline
    bitlinear::InlineTable inl;
    const void *gemm_table; // inside the workspace; null: the weight-streaming kernel runs the sequence
    int gemm_tiles;
    int64_t gemm_total_kb, gemm_min_kb;
    int fronts;             // bit 0: some entry has an RMSNorm in front of the quantiser, bit 1: some entry a SwiGLU
    void *split_scratch;    // inside the workspace; null: the GEMM deals this sequence's tiles whole
    bool trits;             // the weights are in the base-3 format
    bool wide;              // the streaming kernel that runs it: the lockstep one (see decode_is_wide)
};

namespace {
struct SeqLayout {
    size_t acc32, table, lists, gemm, data, total;
    bool use_gemm;
    int64_t gemm_tiles, gemm_total_kb; // CTA tiles and k blocks (tiles x k blocks each) of all matmuls on the GEMM
    int64_t gemm_min_kb;               // the fewest k blocks any of them has
};

inline size_t seq_xq_bytes(int64_t M, int64_t K, bool gemm)
{
    const int64_t rows = (gemm && M < kMinGemmRows) ? kMinGemmRows : M;
    return align_up((size_t)rows * col_tiles(K) * kTileCols, 256);
}

bool seq_layout(const bitlinear_layer_desc *layers, int n, SeqLayout &S, std::vector<size_t> *entry_off)
{
    if (!layers || n <= 0 || n > 65536) return false;
    size_t acc = 0, data = 0;
    uint64_t tiles = 0, gemm_tiles = 0, tokens = 0;
    int64_t max_M = 0;
    for (int i = 0; i < n; ++i)
        if (layers[i].M > max_M) max_M = layers[i].M;
    const bool gemm = use_tcgen05_for(max_M);
    S.use_gemm = gemm;
    for (int i = 0; i < n; ++i) {
        const bitlinear_layer_desc &d = layers[i];
        if (check_shape(d.M, d.N, d.K) != BITLINEAR_OK || d.M < 1) return false;
        tokens += (uint64_t)d.M;
        if (!gemm) acc += align_up((size_t)d.M * d.N * 4, 256);
        tiles += (uint64_t)(row_blocks(d.N) * col_tiles(d.K)); // an upper bound of the work items in either mode
        gemm_tiles += (uint64_t)((d.M + 127) / 128) * (uint64_t)((d.N + 255) / 256); // the same for the GEMM's CTA tiles
        if (entry_off) entry_off->push_back(data);
        data += seq_xq_bytes(d.M, d.K, gemm) + 2 * align_up((size_t)d.M * 4, 256);
    }
    if (tiles > 0xFFFFFFFFull) return false; // the tile sequence is indexed with 32 bits (4 TiB of weights)
    if (tokens > 0x3FFFFFFFull) return false; // tokens (plus the clearing CTAs) index the quantiser's grid with an int
    if (gemm && gemm_tiles > 0x7FFFFFFFull) return false;
    S.gemm_tiles = S.gemm_total_kb = S.gemm_min_kb = 0;
    if (gemm) { // the GEMM's scratch, where the streaming kernel has its int32 scratch
        for (int i = 0; i < n; ++i) {
            S.gemm_tiles += prefill_tile_count(layers[i].M, layers[i].N, max_M);
            S.gemm_total_kb += prefill_kb_count(layers[i].M, layers[i].N, layers[i].K, max_M);
            const int64_t kb = gemm_k_blocks(layers[i].K);
            if (i == 0 || kb < S.gemm_min_kb) S.gemm_min_kb = kb;
        }
        acc = align_up(prefill_scratch_bytes(S.gemm_tiles, S.gemm_total_kb, S.gemm_min_kb, max_M), 256);
    }
    size_t off = sizeof(WorkspaceHeader);
    S.acc32 = off;
    off += acc;
    S.table = off;
    off += align_up((size_t)n * sizeof(DecodeEntry), 256);
    S.lists = off;
    off += align_up(kOwnedListsBytes, 256);
    S.gemm = off;
    if (gemm) off += align_up((size_t)n * kGemmProblemBytes, 256);
    S.data = off;
    off += data;
    S.total = off;
    return true;
}
} // namespace

size_t bitlinear_sequence_workspace_bytes(const bitlinear_layer_desc *layers, int n)
{
    SeqLayout S{};
    if (!seq_layout(layers, n, S, nullptr)) return 0;
    return S.total;
}

namespace {
bitlinear_status sequence_create_impl(const bitlinear_layer_desc *layers, const float *const *gains,
                                      const void *const *ups, float norm_eps, int n, void *workspace,
                                      size_t workspace_bytes, bitlinear_sequence **out, bool trits = false);
}

bitlinear_status bitlinear_sequence_create(const bitlinear_layer_desc *layers, int n, void *workspace,
                                           size_t workspace_bytes, bitlinear_sequence **out)
{
    return sequence_create_impl(layers, nullptr, nullptr, 0.0f, n, workspace, workspace_bytes, out);
}

bitlinear_status bitlinear_sequence_create_trits(const bitlinear_layer_desc *layers, int n, void *workspace,
                                                 size_t workspace_bytes, bitlinear_sequence **out)
{
    if (!layers || n <= 0) return BITLINEAR_ERR_ARG;
    for (int i = 0; i < n; ++i)
        if (layers[i].M > kMaxTritM) return BITLINEAR_ERR_SHAPE;
    return sequence_create_impl(layers, nullptr, nullptr, 0.0f, n, workspace, workspace_bytes, out, true);
}

bitlinear_status bitlinear_sequence_create_rmsnorm(const bitlinear_layer_desc *layers, const float *const *gains,
                                                   float norm_eps, int n, void *workspace, size_t workspace_bytes,
                                                   bitlinear_sequence **out)
{
    if (!gains || !(norm_eps >= 0.0f)) return BITLINEAR_ERR_ARG;
    for (int i = 0; i < n; ++i)
        if (gains[i] && !aligned(gains[i], 16)) return BITLINEAR_ERR_ALIGN;
    return sequence_create_impl(layers, gains, nullptr, norm_eps, n, workspace, workspace_bytes, out);
}

bitlinear_status bitlinear_sequence_create_swiglu(const bitlinear_layer_desc *layers, const float *const *gains,
                                                  const void *const *ups, float norm_eps, int n, void *workspace,
                                                  size_t workspace_bytes, bitlinear_sequence **out)
{
    if (!ups || !(norm_eps >= 0.0f)) return BITLINEAR_ERR_ARG;
    for (int i = 0; i < n; ++i) {
        if (gains && gains[i] && ups[i]) return BITLINEAR_ERR_ARG; // one front per entry
        if ((gains && gains[i] && !aligned(gains[i], 16)) || (ups[i] && !aligned(ups[i], 16))) return BITLINEAR_ERR_ALIGN;
    }
    return sequence_create_impl(layers, gains, ups, norm_eps, n, workspace, workspace_bytes, out);
}

namespace {
// gains == null: no entry is normalised; gains[i] == null: entry i is not; ups likewise (SwiGLU in front)
bitlinear_status sequence_create_impl(const bitlinear_layer_desc *layers, const float *const *gains,
                                      const void *const *ups, float norm_eps, int n, void *workspace,
                                      size_t workspace_bytes, bitlinear_sequence **out, bool trits)
{
    if (!layers || !workspace || !out || n <= 0) return BITLINEAR_ERR_ARG;
    *out = nullptr;
    SeqLayout S{};
    std::vector<size_t> entry_off;
    if (!seq_layout(layers, n, S, &entry_off)) return BITLINEAR_ERR_SHAPE;
    if (!aligned(workspace, 256)) return BITLINEAR_ERR_ALIGN;
    if (workspace_bytes < S.total) return BITLINEAR_ERR_WORKSPACE;
    for (int i = 0; i < n; ++i) {
        const bitlinear_layer_desc &d = layers[i];
        if (!d.packed || !d.gamma || !d.X || !d.Y) return BITLINEAR_ERR_ARG;
        if (!aligned(d.packed, 16) || !aligned(d.X, 16) || !aligned(d.Y, 16) || !aligned(d.gamma, 4))
            return BITLINEAR_ERR_ALIGN;
    }
    if (!device_is_sm100()) return BITLINEAR_ERR_ARCH;
    char *ws = reinterpret_cast<char *>(workspace);

    std::vector<DecodeEntry> table((size_t)n);
    size_t a_off = S.acc32;
    uint32_t tiles = 0;
    int tokens = 0, max_M = 0;
    for (int i = 0; i < n; ++i)
        if ((int)layers[i].M > max_M) max_M = (int)layers[i].M;
    const bool gemm = S.use_gemm;
    uint64_t plain_tiles = 0;
    for (int i = 0; i < n; ++i)
        plain_tiles += (uint64_t)(trits ? trit_row_blocks(layers[i].N) : row_blocks(layers[i].N)) * (uint64_t)col_tiles(layers[i].K);
    const bool wide = !trits && !gemm && decode_is_wide(max_M, plain_tiles); // which streaming kernel serves the sequence
    std::vector<unsigned char> gemm_table(gemm ? (size_t)n * kGemmProblemBytes : 0);
    int gemm_tiles = 0;
    int64_t gemm_kb = 0;
    int fronts = 0;
    for (int i = 0; i < n; ++i) {
        const bitlinear_layer_desc &d = layers[i];
        Layout L{};
        L.acc32 = a_off;
        L.xq = S.data + entry_off[(size_t)i];
        L.beta = L.xq + seq_xq_bytes(d.M, d.K, gemm);
        L.rowsum = L.beta + align_up((size_t)d.M * 4, 256);
        if (!gemm) a_off += align_up((size_t)d.M * d.N * 4, 256);
        DecodeEntry &e = table[(size_t)i];
        fill_entry(e, d.packed, d.gamma, d.X, d.M, d.K, d.N, d.Y, 0, ws, L, trits);
        e.xq_tiled = gemm ? 0 : 1;
        e.gain = gains ? gains[i] : nullptr;
        e.norm_eps = norm_eps;
        e.up = reinterpret_cast<const __nv_bfloat16 *>(ups ? ups[i] : nullptr);
        fronts |= (e.gain ? 1 : 0) | (e.up ? 2 : 0);
        e.tile_begin = tiles;
        e.token_begin = tokens;
        tiles += decode_items(e.NB, e.KB, wide, max_M); // (one kernel serves the whole sequence)
        tokens += (int)d.M;
        if (gemm) {
            int nt = 0;
            if (prefill_table_entry(gemm_table.data() + (size_t)i * kGemmProblemBytes, e.packed, e.gamma, e.Xq, e.beta,
                                    e.rowsum, d.M, d.M < kMinGemmRows ? kMinGemmRows : d.M, d.K, d.N, d.Y, e.qb, max_M,
                                    gemm_tiles, gemm_kb, reinterpret_cast<WorkspaceHeader *>(ws), &nt) != cudaSuccess)
                return BITLINEAR_ERR_CUDA;
            gemm_tiles += nt;
            gemm_kb += (int64_t)nt * gemm_k_blocks(d.K);
        }
    }
    bitlinear_sequence *seq = new (std::nothrow) bitlinear_sequence();
    if (!seq) return BITLINEAR_ERR_ARG;
    seq->workspace = ws;
    seq->lists = reinterpret_cast<OwnedList *>(ws + S.lists);
    seq->n = n;
    seq->tiles = tiles;
    seq->tokens = tokens;
    seq->max_M = max_M;
    seq->max_K = 0;
    for (int i = 0; i < n; ++i)
        if ((int)layers[i].K > seq->max_K) seq->max_K = (int)layers[i].K;
    const size_t clear = gemm ? prefill_scratch_clear_bytes(gemm_tiles, gemm_kb, S.gemm_min_kb, max_M) : 0;
    const bool split = clear > 0;
    seq->zero_bytes = gemm ? S.acc32 + align_up(clear, 256) : S.table; // header and the int32 scratch in use
    seq->dev_table = nullptr;
    seq->gemm_table = nullptr;
    seq->gemm_tiles = gemm_tiles;
    seq->gemm_total_kb = gemm_kb;
    seq->gemm_min_kb = S.gemm_min_kb;
    seq->fronts = fronts;
    seq->trits = trits;
    seq->wide = wide;
    seq->split_scratch = split ? ws + S.acc32 : nullptr;
    if (gemm) {
        if (cudaMemcpy(ws + S.gemm, gemm_table.data(), gemm_table.size(), cudaMemcpyHostToDevice) != cudaSuccess) {
            delete seq;
            return BITLINEAR_ERR_CUDA;
        }
        seq->gemm_table = ws + S.gemm;
    }
    if (n <= kInlineEntries) {
        for (int i = 0; i < n; ++i) seq->inl.e[i] = table[(size_t)i];
    } else {
        if (cudaMemcpy(ws + S.table, table.data(), (size_t)n * sizeof(DecodeEntry), cudaMemcpyHostToDevice) !=
            cudaSuccess) {
            delete seq;
            return BITLINEAR_ERR_CUDA;
        }
        seq->dev_table = reinterpret_cast<const DecodeEntry *>(ws + S.table);
    }
    *out = seq;
    return BITLINEAR_OK;
}
} // namespace

bitlinear_status bitlinear_forward_sequence_stage(const bitlinear_sequence *seq, int stage, void *stream)
{
    if (!seq || stage < 0 || stage > 2) return BITLINEAR_ERR_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    if (stage != 2 &&
        launch_quantize_acts(seq->inl, seq->dev_table, seq->n, seq->tokens, seq->workspace, seq->zero_bytes,
                             seq->fronts, seq->max_K, s) !=
            cudaSuccess)
        return BITLINEAR_ERR_CUDA;
    if (stage != 1) {
        const cudaError_t err =
            seq->gemm_table ? launch_prefill_table(seq->gemm_table, seq->n, seq->gemm_tiles, seq->gemm_total_kb, seq->gemm_min_kb, seq->max_M,
                                                 seq->split_scratch, s)
                            : launch_decode(seq->inl, seq->dev_table, seq->n, seq->tiles, seq->max_M, BITLINEAR_PATH_MMA,
                                            reinterpret_cast<WorkspaceHeader *>(seq->workspace), seq->lists, s, seq->trits, seq->wide);
        if (err != cudaSuccess) return BITLINEAR_ERR_CUDA;
    }
    return BITLINEAR_OK;
}

bitlinear_status bitlinear_forward_sequence(const bitlinear_sequence *seq, void *stream)
{
    return bitlinear_forward_sequence_stage(seq, 0, stream);
}

void bitlinear_sequence_destroy(bitlinear_sequence *seq) { delete seq; }

} // extern "C"
