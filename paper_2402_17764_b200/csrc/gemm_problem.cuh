// What the two tensor-core kernels (the GEMM of prefill_gemm.cu and the weight-stationary form of decode_tc.cu) are told
// about a matmul: its two tensor maps and its parameters, alone as a kernel parameter or as one entry of a table in
// device memory that a launch over the matmuls of a sequence walks.
#pragma once

#include <cuda.h>

#include <cstdint>

#include "internal.cuh"

namespace bitlinear {

constexpr int BM = 128; // tokens per MMA of the GEMM (MMA M, TMEM lanes); a CTA tile has MT of them
constexpr int BN = 256; // features per CTA tile
constexpr int BK = 128; // int8 elements (= bytes) of K per stage

struct Params {
    const float *gamma;
    const float *beta;
    const int32_t *rowsum;
    void *out;
    int M, N, KB; // KB = k blocks of 128 columns
    int tiles_m, tiles_n; // CTA tiles: MT * 128 tokens x 256 features
    int out_i32;
    int out_32b_aligned; // rows of the bf16 output start on 32-byte boundaries
    int tile_begin;      // first CTA tile of this matmul in the launch-wide tile sequence
    long long kb_begin;  // first k block of this matmul in the launch-wide sequence of k blocks (all tiles)
    float qb;            // largest activation code (127, or less for activations of fewer bits)
    int32_t *status;
};

// One matmul of a launch.  A single matmul travels as a kernel parameter; the matmuls of a sequence stand in a table in
// device memory (written once, by the host).
struct alignas(64) GemmProblem {
    CUtensorMap tmap_x, tmap_w;
    Params p;
};
static_assert(sizeof(GemmProblem) == kGemmProblemBytes, "internal.cuh states the size of a table entry");

// The matmul a tile, or a k block of the launch-wide sequence, belongs to.  A CTA's work only goes up, so the search
// resumes where it stopped.
template <bool kTable>
struct ProblemCursor {
    const GemmProblem *table;
    int n, i;
    __device__ ProblemCursor(const GemmProblem &one, const GemmProblem *t, int n_) : table(kTable ? t : &one), n(n_), i(0) {}
    __device__ const GemmProblem &seek(int tile)
    {
        if (kTable) {
            while (i + 1 < n && tile >= table[i + 1].p.tile_begin) ++i;
        }
        return table[i];
    }
    __device__ const GemmProblem &seek_kb(long long pos)
    {
        if (kTable) {
            while (i + 1 < n && pos >= table[i + 1].p.kb_begin) ++i;
        }
        return table[i];
    }
};

// The weight-stationary form for 17 to 64 tokens (decode_tc.cu) over the CTA tiles of `one`, or of the `n` matmuls of a
// device table; the tensor map of the weights must be the swizzled one (tma_host.cuh).  max_M: the largest M of the
// launch (at most 64).
cudaError_t launch_decode_tc(const GemmProblem &one, const GemmProblem *table, int n, int n_tiles, int max_M, cudaStream_t stream);

} // namespace bitlinear
