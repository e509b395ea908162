// Kernel (b): per-token absmax quantisation of bf16 activations to int8
// (Section 2, paragraph after Eq. 3: scaled to [-Qb, Qb] per token, Qb = 127, no zero point; Qb = 2^(b-1) - 1 for
// the b-bit activations the paper's outlook names, with the codes still one per byte).
//
// One CTA per token.  The token is read once with 16-byte loads and kept in registers
// (up to kCache vectors per thread; longer rows re-read the tail, which hits L2), the absmax
// is reduced with warp shuffles, then every element takes one fp32 multiply by 127/beta,
// round-half-to-even, clip, and is stored as int8 together with the row sum of the codes.
// The int8 row is written either as it is ([M, K], for the tensor-core GEMM) or tile by tile
// ([column tile of 64][token][64 bytes], zero beyond K, for the weight-streaming kernel, which fetches the
// activations of a run of column tiles with one bulk copy).
// HBM-bound: 2 B read + 1 B written per element.
//
// With a gain vector the token is normalised first (RMSNorm, one of the "LLaMA-alike components" of Section 2):
// x_k = h_k / sqrt(mean(h^2) + eps) * g_k, then quantised as above.  The normalised values decide integers, so
// the arithmetic is fixed.  The sum of squares is an exact integer, hence order-free: with E the exponent field of the
// token's largest |h| (bfloat16: exponent field e, 8-bit significand m with its hidden bit; e = 0 counts as 1 without
// hidden bit), S = sum_k floor(m_k^2 * 2^30 / 4^(E - e_k)) < 2^63 in 64-bit arithmetic (terms more than 23 binades
// below the largest add nothing), sum h^2 = S * 2^(2E - 298).  Then mean = (float)((double)S / K * 2^(2E - 298)),
// r = 1 / sqrt(max(mean + eps, 2^-126)) with IEEE fp32 add, square root and divide, x_k = (h_k * r) * g_k with two fp32
// multiplications.  A token with an infinity or a NaN gets beta = NaN.
//
// With a second input the token is h_k = silu(gate_k) * up_k (SwiGLU, another of those components: the input of the
// down projection), then quantised as above; the arithmetic is fixed again.  e^-g: z = -g * log2(e), n = z rounded to
// the nearest integer (ties to even), r = fma(n, -ln2_hi, -g), r = fma(n, -ln2_lo, r), p = the Taylor polynomial of
// degree 7 in r by Horner's scheme (seven fused multiply-adds), e^-g = p * 2^n (exact); sigmoid = 1 / (1 + e^-g) with
// one addition and one IEEE reciprocal, taken as 0 below g = -87 and as 1 above 87; h = (g * sigmoid) * u with two
// multiplications.  A token with an infinity or a NaN in either input, or with a product beyond fp32, gets beta = NaN.
#include <cstdlib>

#include "internal.cuh"
#include "ptx.cuh"

namespace bitlinear {

namespace {

constexpr int kThreads = 256;
constexpr int kCacheShort = 4; // 16-byte vectors kept in registers per thread (4 * 8 * 256 = 8192 elements)
constexpr int kCacheLong = 8;  // the same for tokens of 8193 to 16384 elements (plain quantiser only)
constexpr int kSwigluSmemBytes = 56 * 1024; // SwiGLU products of one token in shared memory: 14336 elements

__device__ __forceinline__ uint32_t absmax_bits(uint32_t m, const uint4 &v)
{
    // |bf16| as an unsigned 15-bit integer is monotone in the magnitude
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        m = max(m, w[i] & 0x7FFFu);
        m = max(m, (w[i] >> 16) & 0x7FFFu);
    }
    return m;
}

// Four rounded products -> four int8 in one word.  cvt.pack saturates to [-128, 127]; the products never leave
// [-127, 127] after rounding (|x| <= beta and s = fl(127 / beta), so |x * s| < 127.5), which makes the clip of the
// definition a no-op for finite inputs.
__device__ __forceinline__ uint32_t pack4(float a, float b, float c, float d)
{
    const int qa = __float2int_rn(a), qb = __float2int_rn(b), qc = __float2int_rn(c), qd = __float2int_rn(d);
    // cvt.pack d, a, b, c: d = (c << 16) | (sat8(a) << 8) | sat8(b)
    uint32_t hi, out;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(qd), "r"(qc), "r"(0));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(out) : "r"(qb), "r"(qa), "r"(hi));
    return out;
}

// sigmoid(g) in the fixed fp32 steps stated at the head of this file
__device__ __forceinline__ float sigmoid_steps(float g)
{
    const float t = -g;
    const float tc = fminf(fmaxf(t, -87.0f), 87.0f); // (beyond 87 the result is replaced below)
    const float z = __fmul_rn(tc, 1.44269502162933349609375f); // log2(e)
    // |z| < 2^22: adding 1.5 * 2^23 rounds z to the nearest integer, ties to even, and leaves it in the low bits
    const float shifted = __fadd_rn(z, 12582912.0f);
    const float n = __fadd_rn(shifted, -12582912.0f);
    const int ni = __float_as_int(shifted) - 0x4B400000;
    float r = __fmaf_rn(n, -0.693145751953125f, tc);             // ln2_hi: exact product
    r = __fmaf_rn(n, -1.42860676533018704503775e-06f, r);        // ln2_lo
    float p = __fmaf_rn(r, 1.0f / 5040.0f, 1.0f / 720.0f);
    p = __fmaf_rn(p, r, 1.0f / 120.0f);
    p = __fmaf_rn(p, r, 1.0f / 24.0f);
    p = __fmaf_rn(p, r, 1.0f / 6.0f);
    p = __fmaf_rn(p, r, 0.5f);
    p = __fmaf_rn(p, r, 1.0f);
    p = __fmaf_rn(p, r, 1.0f);
    // p * 2^n by adding n to the exponent field: p lies in [0.7, 1.42] and e^t >= e^-87 is a normal number
    const float e = __int_as_float(__float_as_int(p) + ni * 8388608);
    const float sg = __frcp_rn(__fadd_rn(1.0f, e)); // correctly rounded: the same as 1 / (1 + e)
    // (for g > 87 the steps give e^-87 < 2^-125, 1 + e = 1 and so exactly 1 by themselves)
    return t > 87.0f ? 0.0f : sg;
}

// h = silu(gate) * up of eight elements
__device__ __forceinline__ void swiglu8(const uint4 &gv, const uint4 &uv, float (&h)[8])
{
    const uint32_t gw[4] = {gv.x, gv.y, gv.z, gv.w}, uw[4] = {uv.x, uv.y, uv.z, uv.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const float g0 = __uint_as_float(gw[j] << 16), g1 = __uint_as_float(gw[j] & 0xFFFF0000u);
        const float u0 = __uint_as_float(uw[j] << 16), u1 = __uint_as_float(uw[j] & 0xFFFF0000u);
        h[2 * j] = __fmul_rn(__fmul_rn(g0, sigmoid_steps(g0)), u0);
        h[2 * j + 1] = __fmul_rn(__fmul_rn(g1, sigmoid_steps(g1)), u1);
    }
}

// 8 bf16 -> 8 int8 (two 32-bit words), returns the sum of the eight codes
__device__ __forceinline__ int quant8(const uint4 &v, float s, uint2 &out)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    float p[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        p[2 * i] = __fmul_rn(__uint_as_float(w[i] << 16), s); // one multiply, then round half to even
        p[2 * i + 1] = __fmul_rn(__uint_as_float(w[i] & 0xFFFF0000u), s);
    }
    out.x = pack4(p[0], p[1], p[2], p[3]);
    out.y = pack4(p[4], p[5], p[6], p[7]);
    return __dp4a((int)out.x, 0x01010101, __dp4a((int)out.y, 0x01010101, 0));
}

// kFronts: bit 0, entries may carry a gain vector (RMSNorm in front); bit 1, a second input (SwiGLU in front).  Each
// form is compiled with the branches it needs only, and with the registers they need (a thread keeps 16-byte vectors
// of the token, or, for SwiGLU, the products themselves, in registers between the passes).
// NT threads per token (64, 128, 192 or 256): what a CTA does besides touching its elements (finding its entry,
// three block-wide reductions) is a fixed cost per thread, so short tokens take fewer threads with kCache vectors
// each.  Tokens of more than 8 * kCache * NT elements re-read their tail, which hits L2.
template <int kFronts, int NT, int kCache>
__global__ void __launch_bounds__(NT, ((kFronts & 1) ? 768 : 1024) / NT) quantize_acts_kernel(const __grid_constant__ InlineTable inl,
                                                                 const DecodeEntry *__restrict__ table, int n_entries,
                                                                 int total_tokens, uint4 *zero_ptr, size_t zero_vecs,
                                                                 int h_cap_vecs)
{
    extern __shared__ float4 h_smem[]; // SwiGLU: the products of the first h_cap_vecs vectors of the token
    __shared__ uint32_t s_max[NT / 32];
    __shared__ int s_sum[NT / 32];
    __shared__ unsigned long long s_sq[NT / 32];

    // The matmul that follows may be launched early: it streams weights until it needs what this kernel writes.
    ptx::griddep_launch_dependents();

    // The descriptors are written once, before the first launch (or travel as a kernel parameter), so finding this
    // CTA's token in them (a chain of dependent loads) and fetching its descriptor need not wait for anything.
    const bool clearing = (int)blockIdx.x >= total_tokens;
    const DecodeEntry *tab = table ? table : inl.e;
    // entry that owns this token: the last one whose token_begin <= blockIdx.x
    int lo = 0, hi = clearing ? 0 : n_entries - 1;
    while (lo < hi) {
        int mid = (lo + hi + 1) >> 1;
        if (tab[mid].token_begin <= (int)blockIdx.x) lo = mid; else hi = mid - 1;
    }
    const DecodeEntry e = tab[lo]; // a copy: the fields in use are loaded here

    // This kernel itself may have been launched before the kernel in front of it has ended (the finishing launch of
    // the step before, which lets its dependents in at once): what it reads and overwrites may still be in use.
    ptx::griddep_wait();

    if (clearing) {
        // trailing blocks clear control words and split-K scratch for the matmul that follows
        const size_t n_zero_blocks = gridDim.x - total_tokens;
        for (size_t i = (size_t)(blockIdx.x - total_tokens) * NT + threadIdx.x; i < zero_vecs;
             i += n_zero_blocks * NT)
            zero_ptr[i] = make_uint4(0u, 0u, 0u, 0u);
        return;
    }

    const int t = blockIdx.x - e.token_begin;
    const int K = e.K;
    const int n_vec = K >> 3;
    const uint4 *row = reinterpret_cast<const uint4 *>(e.X + (size_t)t * K);
    // output position of the i-th group of 8 codes of this token, in 8-byte units
    uint2 *out_base = reinterpret_cast<uint2 *>(e.Xq);
    const bool tiled = e.xq_tiled != 0;
    const size_t M = (size_t)e.M;
    auto out_at = [&](int i) -> uint2 & {
        return out_base[tiled ? (((size_t)(i >> 3) * M + (size_t)t) * 8 + (size_t)(i & 7)) : ((size_t)t * n_vec + i)];
    };

    uint4 cache[kCache];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if ((kFronts & 1) && e.gain) {
        // ---- RMSNorm, then the quantiser on the fp32 values (see the head of this file)
        const float4 *gain4 = reinterpret_cast<const float4 *>(e.gain);
        // largest magnitude of the token: |bf16| as a 15-bit integer is monotone, its upper 8 bits are the exponent
        uint32_t top = 0;
#pragma unroll
        for (int c = 0; c < kCache; ++c) {
            const int i = threadIdx.x + c * NT;
            if (i < n_vec) {
                cache[c] = __ldg(row + i);
                top = absmax_bits(top, cache[c]);
            }
        }
        for (int i = threadIdx.x + kCache * NT; i < n_vec; i += NT) top = absmax_bits(top, __ldg(row + i));
        top = __reduce_max_sync(0xffffffffu, top);
        if (lane == 0) s_max[warp] = top;
        __syncthreads();
        top = s_max[0];
#pragma unroll
        for (int w = 1; w < NT / 32; ++w) top = max(top, s_max[w]);
        __syncthreads(); // s_max is used again below
        const bool bad = (top >> 7) == 255u; // an infinity or a NaN somewhere in the token
        const int E = max((int)(top >> 7), 1);

        // h * 2^(149 - E) has the magnitude m * 2^(e - E + 15) (exact; what underflows belongs to terms that are 0),
        // its square is m^2 * 4^(e - E) * 2^30 (exact in fp32: 16 significant bits), and the conversion truncates.
        // 2^(149 - E) is no fp32 when E < 22 (a token of values below 2^-105): then the factor is applied in two steps.
        const bool one_step = E >= 22;
        const float up = __uint_as_float((uint32_t)(one_step ? 276 - E : 254 - E) << 23); // 2^(149 - E) or 2^(127 - E)
        unsigned long long sq = 0;
        auto add_squares = [&](const uint4 &v) {
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float a = __fmul_rn(__uint_as_float(w[i] << 16), up);
                float b = __fmul_rn(__uint_as_float(w[i] & 0xFFFF0000u), up);
                if (!one_step) { // (the same for the whole CTA)
                    a = __fmul_rn(a, 4194304.0f); // 2^22
                    b = __fmul_rn(b, 4194304.0f);
                }
                sq += __float2ull_rz(__fmul_rn(a, a));
                sq += __float2ull_rz(__fmul_rn(b, b));
            }
        };
#pragma unroll
        for (int c = 0; c < kCache; ++c) {
            const int i = threadIdx.x + c * NT;
            if (i < n_vec) add_squares(cache[c]);
        }
        for (int i = threadIdx.x + kCache * NT; i < n_vec; i += NT) add_squares(__ldg(row + i));
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, off);
        if (lane == 0) s_sq[warp] = sq;
        __syncthreads();
        unsigned long long tot = 0;
#pragma unroll
        for (int w = 0; w < NT / 32; ++w) tot += s_sq[w]; // every thread forms the same total
        // mean = S / K * 2^(2E - 298): the power of two as a double built from its exponent field
        const double pow2 = __longlong_as_double((long long)(2 * E - 298 + 1023) << 52);
        const float mean = __double2float_rn(__dmul_rn(__ddiv_rn(__ull2double_rn(tot), (double)K), pow2));
        // (the floor 2^-126 only matters for an all-zero token or one whose mean square underflows fp32: r stays finite)
        const float r = __fdiv_rn(1.0f, __fsqrt_rn(fmaxf(__fadd_rn(mean, e.norm_eps), 1.17549435e-38f)));

        // the eight normalised values of vector i
        auto normalised = [&](const uint4 &v, int i, float (&x)[8]) {
            const float4 g0 = __ldg(gain4 + 2 * i), g1 = __ldg(gain4 + 2 * i + 1);
            const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                x[2 * j] = __fmul_rn(__fmul_rn(__uint_as_float(w[j] << 16), r), g[2 * j]);
                x[2 * j + 1] = __fmul_rn(__fmul_rn(__uint_as_float(w[j] & 0xFFFF0000u), r), g[2 * j + 1]);
            }
        };
        uint32_t mx = 0; // |x| as an unsigned integer is monotone in the magnitude
        auto absmax8 = [&](const float (&x)[8]) {
#pragma unroll
            for (int j = 0; j < 8; ++j) mx = max(mx, __float_as_uint(x[j]) & 0x7FFFFFFFu);
        };
        // the normalised values of the cached vectors stay in registers for the last pass (forming them a second time,
        // gain loads included, was a quarter of the kernel's instructions)
        float xs[kCache][8];
#pragma unroll
        for (int c = 0; c < kCache; ++c) {
            const int i = threadIdx.x + c * NT;
            if (i < n_vec) {
                normalised(cache[c], i, xs[c]);
                absmax8(xs[c]);
            }
        }
        for (int i = threadIdx.x + kCache * NT; i < n_vec; i += NT) {
            float x[8];
            normalised(__ldg(row + i), i, x);
            absmax8(x);
        }
        mx = __reduce_max_sync(0xffffffffu, mx);
        if (lane == 0) s_max[warp] = mx;
        __syncthreads();
        mx = s_max[0];
#pragma unroll
        for (int w = 1; w < NT / 32; ++w) mx = max(mx, s_max[w]);
        const float b = fmaxf(__uint_as_float(mx), kBetaFloor);
        const float s = __fdiv_rn(e.qb, b);

        int sum = 0;
        auto quantise8 = [&](const float (&x)[8], int i) {
            uint2 o;
            o.x = pack4(__fmul_rn(x[0], s), __fmul_rn(x[1], s), __fmul_rn(x[2], s), __fmul_rn(x[3], s));
            o.y = pack4(__fmul_rn(x[4], s), __fmul_rn(x[5], s), __fmul_rn(x[6], s), __fmul_rn(x[7], s));
            out_at(i) = o;
            sum = __dp4a((int)o.x, 0x01010101, __dp4a((int)o.y, 0x01010101, sum));
        };
#pragma unroll
        for (int c = 0; c < kCache; ++c) {
            const int i = threadIdx.x + c * NT;
            if (i < n_vec) quantise8(xs[c], i);
        }
        for (int i = threadIdx.x + kCache * NT; i < n_vec; i += NT) {
            float x[8];
            normalised(__ldg(row + i), i, x);
            quantise8(x, i);
        }
        if (tiled) // the last column tile is filled up with zeros
            for (int i = n_vec + threadIdx.x; i < e.KB * 8; i += NT) out_at(i) = make_uint2(0u, 0u);
        sum = __reduce_add_sync(0xffffffffu, sum);
        if (lane == 0) s_sum[warp] = sum;
        __syncthreads();
        if (threadIdx.x == 0) {
            int total = 0;
#pragma unroll
            for (int w = 0; w < NT / 32; ++w) total += s_sum[w];
            e.beta[t] = bad ? __int_as_float(0x7FC00000) : b;
            e.rowsum[t] = total;
        }
        return;
    }

    if ((kFronts & 2) && e.up) {
        // ---- SwiGLU, then the quantiser on the fp32 values (see the head of this file).  The products wait in shared
        // memory between the two passes (32 registers per thread for them left too few warps resident to cover the
        // dependent arithmetic); each thread reads back what it wrote itself.  The two halves of a vector stand
        // h_cap_vecs apart, so that the 16-byte accesses of a warp are consecutive.  A token longer than the buffer
        // forms the rest a second time.
        const uint4 *urow = reinterpret_cast<const uint4 *>(e.up + (size_t)t * K);
        // largest |h| as an unsigned integer.  An infinity or a NaN in either input makes h an infinity or a NaN (a
        // gate of -inf: -inf * 0), and their bit patterns are the largest.
        uint32_t mx = 0;
        auto form = [&](int i, float (&h)[8]) {
            swiglu8(__ldg(row + i), __ldg(urow + i), h);
#pragma unroll
            for (int j = 0; j < 8; ++j) mx = max(mx, __float_as_uint(h[j]) & 0x7FFFFFFFu);
        };
        for (int i = threadIdx.x; i < n_vec; i += NT) {
            float h[8];
            form(i, h);
            if (i < h_cap_vecs) {
                h_smem[i] = make_float4(h[0], h[1], h[2], h[3]);
                h_smem[h_cap_vecs + i] = make_float4(h[4], h[5], h[6], h[7]);
            }
        }
        mx = __reduce_max_sync(0xffffffffu, mx);
        if (lane == 0) s_max[warp] = mx;
        __syncthreads();
        mx = s_max[0];
#pragma unroll
        for (int w = 1; w < NT / 32; ++w) mx = max(mx, s_max[w]);
        const bool bad = mx >= 0x7F800000u; // an infinity or a NaN in an input, or a product beyond fp32
        const float b = fmaxf(__uint_as_float(mx), kBetaFloor);
        const float s = __fdiv_rn(e.qb, b);

        int sum = 0;
        auto quantise8 = [&](const float (&h)[8], int i) {
            uint2 o;
            o.x = pack4(__fmul_rn(h[0], s), __fmul_rn(h[1], s), __fmul_rn(h[2], s), __fmul_rn(h[3], s));
            o.y = pack4(__fmul_rn(h[4], s), __fmul_rn(h[5], s), __fmul_rn(h[6], s), __fmul_rn(h[7], s));
            out_at(i) = o;
            sum = __dp4a((int)o.x, 0x01010101, __dp4a((int)o.y, 0x01010101, sum));
        };
        for (int i = threadIdx.x; i < n_vec; i += NT) {
            float h[8];
            if (i < h_cap_vecs) {
                const float4 a = h_smem[i], c = h_smem[h_cap_vecs + i];
                h[0] = a.x, h[1] = a.y, h[2] = a.z, h[3] = a.w;
                h[4] = c.x, h[5] = c.y, h[6] = c.z, h[7] = c.w;
            } else {
                swiglu8(__ldg(row + i), __ldg(urow + i), h);
            }
            quantise8(h, i);
        }
        if (tiled) // the last column tile is filled up with zeros
            for (int i = n_vec + threadIdx.x; i < e.KB * 8; i += NT) out_at(i) = make_uint2(0u, 0u);
        sum = __reduce_add_sync(0xffffffffu, sum);
        if (lane == 0) s_sum[warp] = sum;
        __syncthreads();
        if (threadIdx.x == 0) {
            int total = 0;
#pragma unroll
            for (int w = 0; w < NT / 32; ++w) total += s_sum[w];
            e.beta[t] = bad ? __int_as_float(0x7FC00000) : b;
            e.rowsum[t] = total;
        }
        return;
    }

    uint32_t m = 0;
#pragma unroll
    for (int c = 0; c < kCache; ++c) {
        const int i = threadIdx.x + c * NT;
        if (i < n_vec) {
            cache[c] = __ldg(row + i);
            m = absmax_bits(m, cache[c]);
        }
    }
    for (int i = threadIdx.x + kCache * NT; i < n_vec; i += 4 * NT) { // four loads in flight
        uint4 v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = (i + j * NT < n_vec) ? __ldg(row + i + j * NT) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int j = 0; j < 4; ++j) m = absmax_bits(m, v[j]);
    }

    m = __reduce_max_sync(0xffffffffu, m);
    if (lane == 0) s_max[warp] = m;
    __syncthreads();
    m = s_max[0];
#pragma unroll
    for (int w = 1; w < NT / 32; ++w) m = max(m, s_max[w]);

    const float amax = __uint_as_float(m << 16);
    const float b = fmaxf(amax, kBetaFloor);
    const float s = __fdiv_rn(e.qb, b); // one IEEE divide per token

    int sum = 0;
#pragma unroll
    for (int c = 0; c < kCache; ++c) {
        const int i = threadIdx.x + c * NT;
        if (i < n_vec) {
            uint2 o;
            sum += quant8(cache[c], s, o);
            out_at(i) = o;
        }
    }
    for (int i = threadIdx.x + kCache * NT; i < n_vec; i += 4 * NT) {
        uint4 v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = (i + j * NT < n_vec) ? __ldg(row + i + j * NT) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (i + j * NT < n_vec) {
                uint2 o;
                sum += quant8(v[j], s, o);
                out_at(i + j * NT) = o;
            }
        }
    }
    if (tiled) // the last column tile is filled up with zeros
        for (int i = n_vec + threadIdx.x; i < e.KB * 8; i += NT) out_at(i) = make_uint2(0u, 0u);
    sum = __reduce_add_sync(0xffffffffu, sum);
    if (lane == 0) s_sum[warp] = sum;
    __syncthreads();
    if (threadIdx.x == 0) {
        int tot = 0;
#pragma unroll
        for (int w = 0; w < NT / 32; ++w) tot += s_sum[w];
        e.beta[t] = b;
        e.rowsum[t] = tot;
    }
}

__global__ void __launch_bounds__(kThreads) retile_acts_kernel(const int8_t *__restrict__ Xq, int M, int K, int KB,
                                                               int8_t *__restrict__ tiled)
{
    const int t = blockIdx.x;
    const uint2 *row = reinterpret_cast<const uint2 *>(Xq + (size_t)t * K);
    uint2 *out = reinterpret_cast<uint2 *>(tiled);
    for (int i = threadIdx.x; i < KB * 8; i += kThreads)
        out[((size_t)(i >> 3) * M + t) * 8 + (i & 7)] = (i < (K >> 3)) ? __ldg(row + i) : make_uint2(0u, 0u);
}

} // namespace

cudaError_t launch_retile_acts(const int8_t *Xq, int64_t M, int64_t K, int8_t *tiled, cudaStream_t stream)
{
    if (M == 0) return cudaSuccess;
    const int KB = (int)((K + kTileCols - 1) / kTileCols);
    retile_acts_kernel<<<(unsigned)M, kThreads, 0, stream>>>(Xq, (int)M, (int)K, KB, tiled);
    return cudaGetLastError();
}

cudaError_t launch_quantize_acts(const InlineTable &inl, const DecodeEntry *table, int n_entries, int total_tokens,
                                 void *zero_ptr, size_t zero_bytes, int fronts, int max_K, cudaStream_t stream)
{
    // threads per token: the smallest count whose register caches hold the longest token
    const int n_vec = max_K >> 3;
    // (longer tokens re-read their tail, which hits L2: CTAs of 512 and 1024 threads measured slower)
    static const int counts[4] = {64, 128, 192, 256};
    int nt = 256;
    for (int c : counts)
        if (n_vec <= c * kCacheShort) {
            nt = c;
            break;
        }
    // SwiGLU: room in shared memory for the products of a token (at most kSwigluSmemBytes: four CTAs per SM)
    int h_cap_vecs = 0;
    size_t dyn_smem = 0;
    if (fronts & 2) {
        h_cap_vecs = n_vec < kSwigluSmemBytes / 32 ? n_vec : kSwigluSmemBytes / 32;
        dyn_smem = (size_t)h_cap_vecs * 32;
    }
    const size_t zero_vecs = zero_bytes / 16;
    int zero_blocks = 0;
    if (zero_vecs > 0) {
        zero_blocks = (int)((zero_vecs + (size_t)nt * 4 - 1) / ((size_t)nt * 4));
        const int cap = sm_count() * 1024 / nt;
        if (zero_blocks > cap) zero_blocks = cap;
        if (zero_blocks < 1) zero_blocks = 1;
    }
    const int grid = total_tokens + zero_blocks;
    if (grid == 0) return cudaSuccess;
    uint4 *zp = reinterpret_cast<uint4 *>(zero_ptr);
    // A programmatic dependent of whatever stands in front of it on the stream: behind the finishing launch of a
    // step before, the CTAs are resident and waiting when that launch ends (BITLINEAR_QUANTISER_EARLY_LAUNCH=0: off).
    static const bool early = [] {
        const char *v = std::getenv("BITLINEAR_QUANTISER_EARLY_LAUNCH");
        return !(v && *v == '0');
    }();
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.dynamicSmemBytes = dyn_smem;
    cfg.stream = stream;
    cfg.attrs = &attr;
    cfg.numAttrs = early ? 1 : 0;
#define BITLINEAR_LAUNCH_QUANTISER(FRONTS, NT_) \
    do { \
        if (FRONTS & 2) { \
            static bool attr_set[64] = {false}; \
            int dev = 0; \
            cudaGetDevice(&dev); \
            if (dev >= 0 && dev < 64 && !attr_set[dev]) { \
                cudaError_t e = cudaFuncSetAttribute(quantize_acts_kernel<FRONTS, NT_, kCacheShort>, \
                                                     cudaFuncAttributeMaxDynamicSharedMemorySize, kSwigluSmemBytes); \
                if (e != cudaSuccess) return e; \
                attr_set[dev] = true; \
            } \
        } \
        cfg.blockDim = dim3(NT_); \
        cudaError_t le = cudaLaunchKernelEx(&cfg, quantize_acts_kernel<FRONTS, NT_, kCacheShort>, inl, table, n_entries, \
                                            total_tokens, zp, zero_vecs, h_cap_vecs); \
        if (le != cudaSuccess) return le; \
    } while (0)
#define BITLINEAR_LAUNCH_BOTH(NT_) \
    do { \
        switch (fronts & 3) { \
        case 0: BITLINEAR_LAUNCH_QUANTISER(0, NT_); break; \
        case 1: BITLINEAR_LAUNCH_QUANTISER(1, NT_); break; \
        case 2: BITLINEAR_LAUNCH_QUANTISER(2, NT_); break; \
        default: BITLINEAR_LAUNCH_QUANTISER(3, NT_); break; \
        } \
    } while (0)
    if ((fronts & 3) == 0 && n_vec > 256 * kCacheShort && n_vec <= 256 * kCacheLong) {
        // long tokens of the plain quantiser: twice the vectors in registers, so that the token is read once
        // (CTAs of 512 threads with four vectors each were slower: 4.7 against 5.8 TB/s on 8192 x 13824)
        cfg.blockDim = dim3(256);
        cudaError_t le = cudaLaunchKernelEx(&cfg, quantize_acts_kernel<0, 256, kCacheLong>, inl, table, n_entries, total_tokens,
                                            zp, zero_vecs, h_cap_vecs);
        return le != cudaSuccess ? le : cudaGetLastError();
    }
    switch (nt) {
    case 64: BITLINEAR_LAUNCH_BOTH(64); break;
    case 128: BITLINEAR_LAUNCH_BOTH(128); break;
    case 192: BITLINEAR_LAUNCH_BOTH(192); break;
    default: BITLINEAR_LAUNCH_BOTH(256); break;
    }
#undef BITLINEAR_LAUNCH_BOTH
#undef BITLINEAR_LAUNCH_QUANTISER
    return cudaGetLastError();
}

} // namespace bitlinear
