// Host-visible interface of the tensor-core GEMM kernel.
#pragma once

#include <cstdint>
#include <cuda.h>
#include <cuda_runtime.h>

#include "../../include/mpgemmfi.h"

namespace mpg {

struct GemmParams {
    int dtype, M, N, K;
    int detect_mode, n_faults;
    int tiles_m, tiles_n, num_tiles, num_kt;
    int wpr;        // bitmap words per row = ceil(N / 32)
    int c_vec_ok;   // C rows allow 16-byte vector stores
    const void *A;
    const void *Bt;
    float *C;
    const mpgemmfi_site *sites;
    uint32_t *flags;
};

// shared-memory pipeline depth used for an output tile that is bn columns wide
int gemm_stage_count(int bn);

// bn in {64, 128, 256}: width of the output tile; tm_a / tm_b must have been encoded with
// boxes of (128 bytes x 128 rows) and (128 bytes x bn rows), 128-byte swizzle.
cudaError_t launch_gemm(int bn, const CUtensorMap &tm_a, const CUtensorMap &tm_b, const GemmParams &p, int grid,
                        cudaStream_t stream);

}  // namespace mpg
