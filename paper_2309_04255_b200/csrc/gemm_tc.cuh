// Host-visible interface of the tensor-core skinny GEMM (gemm_tc.cu).
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace llmcad {

struct TcGemmParams {
    int n_tiles;        // tiles of 128 output features
    int kb_per_tile;    // 64-wide k-blocks per tile
    int n_pad;          // tree nodes padded to a multiple of 16 (the MMA N)
    int dual;           // 1: every tile carries a gate and an up accumulator (SwiGLU)
    int up_row_offset;  // row of the first up-projection row in the packed [2f][d] matrix
    int units_per_cta;  // (tile, k-block) units per CTA of the persistent grid
    int stages;         // depth of the shared-memory ring
    int tmem_cols;      // allocated TMEM columns (power of two)
    float *partials;    // [grid][2 slots][n_acc][n_pad][128] fp32 partial tiles
    uint32_t *tickets;  // [n_tiles][4] arrivals per (tile, 32-row group); zero between launches
    int32_t *status;
    unsigned long long *trace;  // optional [grid][16] timeline in ns (nullptr: off)
    EpiParams ep;
};

// Tensor map over a row-major bf16 matrix [rows][cols] with a box of 64 columns x box_rows rows
// and 128-byte swizzle. cols must be a multiple of 8 and base 16-byte aligned.
bool make_tensor_map_bf16(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows);

size_t gemm_tc_partial_floats(int n_sms, int max_n_pad);

cudaError_t launch_gemm_tc(const CUtensorMap &tm_w, const CUtensorMap &tm_x, int n_in, int n_pad, int n_sms,
                           float *partials, uint32_t *flags, uint32_t epoch, int32_t *status, const EpiParams &ep,
                           cudaStream_t st, unsigned long long *trace = nullptr);

}  // namespace llmcad
