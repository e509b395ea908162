// Kernel (a): absmean weight quantisation (Section 2, Eq. 1-3) and 2-bit packing.
//
// Three launches on the caller's stream:
//   1. clear 32 bytes of scratch (the head of the output buffer itself),
//   2. exact sum of |W| in 2^-64 fixed point, 128-bit integer, order-free; the last block
//      to finish turns it into gamma,
//   3. ternarise with round-half-to-even and write the interleaved 2-bit tiles.
// HBM-bound: two reads of the fp32 matrix (8 B per weight) and 0.25 B written per weight.
#include "exact_sum.cuh"
#include "internal.cuh"

namespace bitlinear {

namespace {

// scratch words (unsigned long long): [0] sum.lo  [1] sum.hi  [2] blocks done  [3] range violation flag
__global__ void __launch_bounds__(256) absmean_kernel(const float4 *__restrict__ W4, size_t n_vec,
                                                      double count, unsigned long long *scratch,
                                                      float *__restrict__ gamma)
{
    U128 acc = {0ull, 0ull};
    uint32_t bad = 0;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec; i += (size_t)gridDim.x * blockDim.x) {
        float4 v = __ldg(W4 + i);
        const float f[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t mag = __float_as_uint(f[j]) & 0x7FFFFFFFu;
            if ((mag >> 23) >= 151u) { bad = 1; continue; }
            unsigned long long lo, hi;
            fix64(mag, lo, hi);
            add128(acc, lo, hi);
        }
    }
    // warp reduction
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        unsigned long long lo = __shfl_xor_sync(0xffffffffu, acc.lo, off);
        unsigned long long hi = __shfl_xor_sync(0xffffffffu, acc.hi, off);
        add128(acc, lo, hi);
        bad |= __shfl_xor_sync(0xffffffffu, bad, off);
    }
    __shared__ U128 warp_sum[8];
    __shared__ uint32_t warp_bad[8];
    __shared__ bool is_last;
    int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) { warp_sum[warp] = acc; warp_bad[warp] = bad; }
    __syncthreads();
    if (threadIdx.x == 0) {
        U128 tot = {0ull, 0ull};
        uint32_t b = 0;
        for (int w = 0; w < 8; ++w) { add128(tot, warp_sum[w].lo, warp_sum[w].hi); b |= warp_bad[w]; }
        // 128-bit atomic add as two 64-bit ones: the number of carries out of the low word
        // does not depend on the order in which blocks arrive.
        unsigned long long old = atomicAdd(&scratch[0], tot.lo);
        unsigned long long carry = (old + tot.lo < old) ? 1ull : 0ull;
        atomicAdd(&scratch[1], tot.hi + carry);
        if (b) atomicOr(&scratch[3], 1ull);
        __threadfence();
        unsigned long long ticket = atomicAdd(&scratch[2], 1ull);
        is_last = (ticket == (unsigned long long)gridDim.x - 1ull);
    }
    __syncthreads();
    if (is_last && threadIdx.x == 0) {
        __threadfence();
        unsigned long long lo = atomicAdd(&scratch[0], 0ull);
        unsigned long long hi = atomicAdd(&scratch[1], 0ull);
        unsigned long long flag = atomicAdd(&scratch[3], 0ull);
        double sum = __dmul_rn(__dadd_rn(__dmul_rn(__ull2double_rn(hi), 18446744073709551616.0), __ull2double_rn(lo)),
                               1.0 / 18446744073709551616.0);
        double mean = __ddiv_rn(sum, count);
        *gamma = flag ? __int_as_float(0x7FC00000) : __double2float_rn(mean);
    }
}

// One warp per tile of 64 rows x 64 columns (1 KiB = two slabs of 512 bytes).  Lane (g = lane / 4,
// tq = lane % 4) owns rows 16 f + 8 h + g (f = 0..3, h = 0, 1) and columns 16 tq .. 16 tq + 15 of the tile:
// the code of row (f, h), column 16 tq + 8 s + 4 hi + b goes to slab s, word 2 hi + h, byte b, bits 2f, 2f+1
// of the lane's 16 bytes.  Rows >= N and columns >= K hold code 1 (weight 0).
__global__ void __launch_bounds__(256) ternarize_pack_kernel(const float *__restrict__ W, int N, int K, int NB, int KB,
                                                             float eps, const float *__restrict__ gamma,
                                                             uint4 *__restrict__ packed)
{
    const long long n_tiles = (long long)NB * KB;
    const int lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3;
    const float denom = __fadd_rn(*gamma, eps); // Eq. 1: gamma + eps
    for (long long tile = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); tile < n_tiles;
         tile += (long long)gridDim.x * (blockDim.x >> 5)) {
        const int rb = (int)(tile / KB), kb = (int)(tile % KB);
        uint32_t words[2][4] = {{0u, 0u, 0u, 0u}, {0u, 0u, 0u, 0u}};
        const int col0 = kb * kTileCols + 16 * tq;
#pragma unroll
        for (int f = 0; f < 4; ++f) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int n = rb * kTileRows + 16 * f + 8 * h + g;
                const float *row = W + (size_t)n * K;
#pragma unroll
                for (int v = 0; v < 4; ++v) { // four float4 = 16 columns; v = 2 s + hi
                    const int col = col0 + 4 * v;
                    uint32_t codes = 0x01010101u; // padding: weight 0
                    if (n < N && col < K) {
                        float4 w = __ldg(reinterpret_cast<const float4 *>(row + col));
                        const float x[4] = {w.x, w.y, w.z, w.w};
                        codes = 0;
#pragma unroll
                        for (int b = 0; b < 4; ++b) {
                            int t = __float2int_rn(__fdiv_rn(x[b], denom)); // round half to even (Eq. 2)
                            t = max(-1, min(1, t));
                            codes |= (uint32_t)(t + 1) << (8 * b);
                        }
                    }
                    words[v >> 1][2 * (v & 1) + h] |= codes << (2 * f);
                }
            }
        }
        packed[tile * 64 + lane] = make_uint4(words[0][0], words[0][1], words[0][2], words[0][3]);
        packed[tile * 64 + 32 + lane] = make_uint4(words[1][0], words[1][1], words[1][2], words[1][3]);
    }
}

// The same for the base-3 format: one warp per tile of 80 rows x 64 columns (still 1 KiB).  The byte positions are
// those above; a byte holds the codes of the FIVE rows 16 f + 8 h + g, f = 0..4, as the number sum_f 3^f code_f.
__global__ void __launch_bounds__(256) ternarize_pack_trits_kernel(const float *__restrict__ W, int N, int K, int NB, int KB,
                                                                   float eps, const float *__restrict__ gamma,
                                                                   uint4 *__restrict__ packed)
{
    const long long n_tiles = (long long)NB * KB;
    const int lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3;
    const float denom = __fadd_rn(*gamma, eps); // Eq. 1: gamma + eps
    for (long long tile = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); tile < n_tiles;
         tile += (long long)gridDim.x * (blockDim.x >> 5)) {
        const int rb = (int)(tile / KB), kb = (int)(tile % KB);
        uint32_t words[2][4] = {{0u, 0u, 0u, 0u}, {0u, 0u, 0u, 0u}};
        const int col0 = kb * kTileCols + 16 * tq;
        uint32_t weight = 1u; // 3^f
#pragma unroll
        for (int f = 0; f < 5; ++f) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int n = rb * 80 + 16 * f + 8 * h + g;
                const float *row = W + (size_t)n * K;
#pragma unroll
                for (int v = 0; v < 4; ++v) { // four float4 = 16 columns; v = 2 s + hi
                    const int col = col0 + 4 * v;
                    uint32_t codes = 0x01010101u; // padding: weight 0
                    if (n < N && col < K) {
                        float4 w = __ldg(reinterpret_cast<const float4 *>(row + col));
                        const float x[4] = {w.x, w.y, w.z, w.w};
                        codes = 0;
#pragma unroll
                        for (int b = 0; b < 4; ++b) {
                            int t = __float2int_rn(__fdiv_rn(x[b], denom)); // round half to even (Eq. 2)
                            t = max(-1, min(1, t));
                            codes |= (uint32_t)(t + 1) << (8 * b);
                        }
                    }
                    words[v >> 1][2 * (v & 1) + h] += codes * weight; // (no byte exceeds 242: no carry between bytes)
                }
            }
            weight *= 3u;
        }
        packed[tile * 64 + lane] = make_uint4(words[0][0], words[0][1], words[0][2], words[0][3]);
        packed[tile * 64 + 32 + lane] = make_uint4(words[1][0], words[1][1], words[1][2], words[1][3]);
    }
}

__global__ void __launch_bounds__(256) unpack_trits_kernel(const uint8_t *__restrict__ packed, int N, int K, int KB,
                                                           int8_t *__restrict__ T)
{
    const size_t total = (size_t)N * K;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
        const int n = (int)(idx / K), k = (int)(idx % K);
        const size_t tile = (size_t)(n / 80) * KB + k / kTileCols;
        const int r = n % 80, c = k % kTileCols;
        const int f = r / 16, h = (r % 16) / 8, g = r % 8;
        const int tq = c / 16, s = (c % 16) / 8, hi = (c % 8) / 4, b = c % 4;
        int v = packed[tile * kTileBytes + s * 512 + (4 * g + tq) * 16 + 4 * (2 * hi + h) + b];
        for (int i = 0; i < f; ++i) v /= 3;
        T[idx] = (int8_t)(v % 3 - 1);
    }
}

__global__ void __launch_bounds__(256) unpack_kernel(const uint8_t *__restrict__ packed, int N, int K, int KB,
                                                     int8_t *__restrict__ T)
{
    const size_t total = (size_t)N * K;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
        const int n = (int)(idx / K), k = (int)(idx % K);
        const size_t tile = (size_t)(n / kTileRows) * KB + k / kTileCols;
        const int r = n % kTileRows, c = k % kTileCols;
        const int f = r / 16, h = (r % 16) / 8, g = r % 8;
        const int tq = c / 16, s = (c % 16) / 8, hi = (c % 8) / 4, b = c % 4;
        const uint8_t byte = packed[tile * kTileBytes + s * 512 + (4 * g + tq) * 16 + 4 * (2 * hi + h) + b];
        T[idx] = (int8_t)(((byte >> (2 * f)) & 3) - 1);
    }
}

// Counts the 2-bit fields of a packed buffer that hold 3, the code no weight has (over the whole buffer, padding
// included: every field there is 1).  A field is 3 exactly where both of its bits are set.
__global__ void __launch_bounds__(256) count_bad_codes_kernel(const uint4 *__restrict__ packed, size_t n_vec,
                                                              int32_t *__restrict__ bad)
{
    int found = 0;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec; i += (size_t)gridDim.x * blockDim.x) {
        const uint4 v = __ldg(packed + i);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) found += __popc(w[j] & (w[j] >> 1) & 0x55555555u);
    }
    found = __reduce_add_sync(0xffffffffu, found);
    if ((threadIdx.x & 31) == 0 && found) atomicAdd(bad, found);
}

} // namespace

cudaError_t launch_count_bad_codes(const void *packed, size_t bytes, int32_t *bad, cudaStream_t stream)
{
    cudaError_t err = cudaMemsetAsync(bad, 0, sizeof(int32_t), stream);
    if (err != cudaSuccess) return err;
    const size_t n_vec = bytes / 16;
    size_t blocks = (n_vec + 255) / 256;
    if (blocks > (size_t)sm_count() * 8) blocks = (size_t)sm_count() * 8;
    count_bad_codes_kernel<<<(int)blocks, 256, 0, stream>>>(reinterpret_cast<const uint4 *>(packed), n_vec, bad);
    return cudaGetLastError();
}

cudaError_t launch_absmean_and_pack(const float *W, int64_t N, int64_t K, float eps, void *packed, float *gamma,
                                    cudaStream_t stream, bool trits)
{
    cudaError_t err = cudaMemsetAsync(packed, 0, 32, stream);
    if (err != cudaSuccess) return err;
    const size_t n_vec = (size_t)N * K / 4;
    int blocks = (int)((n_vec + 255) / 256);
    const int cap = sm_count() * 8;
    if (blocks > cap) blocks = cap;
    absmean_kernel<<<blocks, 256, 0, stream>>>(reinterpret_cast<const float4 *>(W), n_vec, (double)(N * K),
                                               reinterpret_cast<unsigned long long *>(packed), gamma);
    err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    const int KB = (int)((K + kTileCols - 1) / kTileCols);
    const int NB = trits ? (int)((N + 79) / 80) : (int)((N + kTileRows - 1) / kTileRows);
    const long long n_tiles = (long long)NB * KB;
    long long pblocks = (n_tiles + 7) / 8;
    if (pblocks > (long long)sm_count() * 16) pblocks = (long long)sm_count() * 16;
    if (trits)
        ternarize_pack_trits_kernel<<<(int)pblocks, 256, 0, stream>>>(W, (int)N, (int)K, NB, KB, eps, gamma,
                                                                      reinterpret_cast<uint4 *>(packed));
    else
        ternarize_pack_kernel<<<(int)pblocks, 256, 0, stream>>>(W, (int)N, (int)K, NB, KB, eps, gamma,
                                                                reinterpret_cast<uint4 *>(packed));
    return cudaGetLastError();
}

cudaError_t launch_unpack(const void *packed, int64_t N, int64_t K, int8_t *T, cudaStream_t stream, bool trits)
{
    const int KB = (int)((K + kTileCols - 1) / kTileCols);
    size_t total = (size_t)N * K;
    size_t blocks = (total + 255) / 256;
    if (blocks > (size_t)sm_count() * 32) blocks = (size_t)sm_count() * 32;
    if (trits)
        unpack_trits_kernel<<<(int)blocks, 256, 0, stream>>>(reinterpret_cast<const uint8_t *>(packed), (int)N, (int)K, KB, T);
    else
        unpack_kernel<<<(int)blocks, 256, 0, stream>>>(reinterpret_cast<const uint8_t *>(packed), (int)N, (int)K, KB, T);
    return cudaGetLastError();
}

} // namespace bitlinear
