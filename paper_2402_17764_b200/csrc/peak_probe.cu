// Measurement aid: what the int8 tensor cores of this GPU sustain when nothing but MMAs is issued.
//
// The prefill matmul (Section 3, "Energy": the matrix multiplication dominates) is reported as a fraction of the int8
// tensor peak.  The nominal figure is a datasheet number at a clock the part does not hold under load, so the benchmark
// measures the ceiling itself, in the same run: one CTA per SM puts one activation-shaped tile (128 x 128 bytes, s8) and
// one weight-shaped tile (256 x 128 bytes, u8) of pseudo-random bytes into shared memory ONCE, and then a single thread
// issues tcgen05.mma kind::i8 (128 x 256 x 32) back to back on them into two TMEM accumulators -- no loads, no
// expansion, no epilogue inside the loop.  2 * 128 * 256 * 32 integer operations per MMA, four MMAs per iteration.
// Operand bytes are random rather than zero because the power the multipliers draw, and with it the clock the part
// settles at, depends on the data.
#include "internal.cuh"
#include "ptx.cuh"

namespace bitlinear {

namespace {

using namespace ptx;

constexpr int kProbeThreads = 128;
constexpr uint32_t kProbeABytes = 128 * 128; // 128 tokens x 128 bytes of K
constexpr uint32_t kProbeBBytes = 256 * 128; // 256 features x 128 bytes of K
constexpr uint32_t kProbeSmem = 1024 + kProbeABytes + kProbeBBytes + 64;

__device__ __forceinline__ uint32_t mix(uint32_t x)
{
    x ^= x >> 16;
    x *= 0x7feb352dU;
    x ^= x >> 15;
    x *= 0x846ca68bU;
    x ^= x >> 16;
    return x;
}

__global__ void __launch_bounds__(kProbeThreads, 1) int8_issue_probe_kernel(int iters, int32_t *status, uint32_t limit_us)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u; // swizzled tiles need 1024-byte alignment
    uint8_t *smem = smem_raw + (base - raw);
    uint64_t *done = reinterpret_cast<uint64_t *>(smem + kProbeABytes + kProbeBBytes);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(done + 1);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    // operand bytes: activations in [-127, 127], weights as the expander writes them (code * 4^f, code 0..2)
    uint32_t *words = reinterpret_cast<uint32_t *>(smem);
    for (uint32_t i = threadIdx.x; i < (kProbeABytes + kProbeBBytes) / 4; i += kProbeThreads) {
        uint32_t r = mix(i * 2654435761u + blockIdx.x);
        if (i >= kProbeABytes / 4) {
            const uint32_t f = (i >> 9) & 3u; // sixteen rows of 128 bytes share a field
            uint32_t c = r & 0x03030303u;     // two random bits per byte
            c -= (c >> 1) & c;                // 3 -> 2: codes 0, 1, 2
            r = c << (2 * f);
        }
        words[i] = r;
    }
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(done), 1);
        *abort_flag = 0;
        fence_mbar_init();
    }
    fence_proxy_async_smem(); // generic-proxy writes -> visible to the tensor core
    if (threadIdx.x < 32) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (threadIdx.x == 0) {
        const uint32_t idesc = idesc_i8(128, 256, /*a_signed=*/1, /*b_signed=*/0);
        const uint64_t a_desc = smem_desc_k_sw128(base), b_desc = smem_desc_k_sw128(base + kProbeABytes);
        for (int it = 0; it < iters; ++it) {
            const uint32_t d = tmem_base + (uint32_t)(it & 1) * 256u;
            // a fresh sum every 64 iterations per accumulator: |acc| <= 127 * 170 * 128 * 64 < 2^31
            uint32_t accumulate = ((it >> 1) & 63) ? 1u : 0u;
#pragma unroll
            for (int k4 = 0; k4 < 4; ++k4) {
                mma_i8_ss(d, a_desc + 2 * k4, b_desc + 2 * k4, idesc, accumulate);
                accumulate = 1u;
            }
        }
        mma_commit(smem_u32(done));
        if (!mbar_wait_bounded(smem_u32(done), 0, abort_flag, limit_us)) atomicExch(status, (int32_t)BITLINEAR_ERR_TIMEOUT);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x < 32) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
}

} // namespace

cudaError_t launch_int8_issue_probe(int iters, int32_t *status, int *ctas, cudaStream_t stream)
{
    static bool attr_set[64] = {false};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(int8_issue_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kProbeSmem);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    const int n = sm_count();
    if (ctas) *ctas = n;
    // the whole loop runs behind ONE wait: iters MMAs of 128 clocks each must fit the limit with room to spare
    int8_issue_probe_kernel<<<n, kProbeThreads, kProbeSmem, stream>>>(iters, status, ptx::kWaitLimitUs);
    return cudaGetLastError();
}

} // namespace bitlinear
