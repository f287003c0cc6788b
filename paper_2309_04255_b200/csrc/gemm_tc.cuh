// Host-visible interface of the tensor-core skinny GEMM (gemm_tc.cu): a weight-streaming kernel that
// leaves the accumulators of every tile segment in a workspace, and a finishing kernel that adds the
// segments of each tile and applies the fused epilogue.
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace llmcad {

// One GEMM: D[n_out][n] = W[n_out][n_in] X[n][n_in]^T followed by its fused epilogue.
struct GemmDesc {
    int n_tiles;        // tiles of 128 output features
    int kb_per_tile;    // 64-wide k-blocks per tile
    int pair_k;         // k-blocks per ring item (1 or 2), set by the launcher
    int halves;         // 2: every tile carries a gate and an up accumulator (SwiGLU), else 1
    int up_row_offset;  // row of the first up-projection row in the packed [2f][d] matrix
    int items_per_cta;  // ring items ((tile, k-block, half) triples) per CTA of the streaming grid
    int grid;           // CTAs of the streaming grid
    const uint8_t *w_tiled;  // weights as a sequence of pre-swizzled 16 KB tiles [tile][k-block] (see pack.cu),
                             // or nullptr: row-major weights through the tensor map
    int up_tile_offset;      // first tile of the up projection in the tiled sequence
    int w4;                  // 1: w_tiled holds INT4 tiles (pack.cu, 4224 bytes per tile and k-block) that the kernel
                             // turns into bf16 tiles in shared memory on their way to the MMA
    EpiParams ep;
};

struct GemmMaps {
    CUtensorMap w;  // weight matrix, box 64 x 128 rows (row-major weights only)
    CUtensorMap x;  // the activation matrix, box 64 x n_pad rows x planes (hi, lo)
};

struct GemmParams {
    int n_pad;          // tree nodes padded to a multiple of 16
    int comp;           // 1: activations come as hi + lo planes; the MMA N is 2 * n_pad and the two columns of a node are added
    int acc_bufs;       // accumulator buffers in TMEM: 2, or 1 when 2 x (gate | up) x MMA N exceeds the 512 columns
    int stages;         // depth of the shared-memory ring (INT4 weights: of the ring of expanded weight items)
    int pstages;        // INT4 weights: depth of the ring of packed tiles that feeds it
    int astages;        // INT4 weights: depth of the ring of activation items (with bf16 weights they share the weights' stages)
    int tmem_cols;      // allocated TMEM columns (power of two)
    float *partials;    // segment slots [n_tiles + grid][4 row groups][halves][n_pad][32 rows] fp32: the segment of
                        // tile t held by CTA c sits in slot t + c
    int32_t *status;
    unsigned long long *trace;  // optional [256][16] timeline in ns of this GEMM (nullptr: off)
    int withhold_act;   // self-test of the wait limit: the activation copies are never issued
    uint64_t wait_limit_ns;   // bound of every device-side wait of the launch
    // hand-over counters (common.cuh): the streaming kernel waits for `dep` (its input is final, the workspace is
    // free), its four dump warps arrive at s_done; the finishing kernel waits for s_done (4 x grid arrivals) and
    // every CTA of it arrives at f_done (f_grid arrivals, set by the launcher). Null: grid dependencies instead.
    const uint32_t *dep_ctr;
    uint32_t dep_target;
    uint32_t *s_done, *f_done;
    int f_grid;
    GemmDesc g;
};

// Tensor map over a row-major bf16 matrix [rows][cols] with a box of 64 columns x box_rows rows
// and 128-byte swizzle. cols must be a multiple of 8 and base 16-byte aligned.
bool make_tensor_map_bf16(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows);

// Tensor map over `planes` (1 or 2) row-major bf16 matrices [rows][cols] that lie plane_rows rows
// apart, with a box of 64 columns x box_rows rows x planes: one copy brings the hi and the lo tile
// of an activation k-block, one after the other, into shared memory. Rows beyond `rows` read as zero.
bool make_act_map_bf16(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows, uint32_t planes,
                       uint64_t plane_rows);
// Any three-dimensional bf16 tensor with 128-byte swizzle and zero fill outside its bounds: dims and box
// innermost first, strides (bytes) of dimensions 1 and 2.
bool make_tensor_map_bf16_3d(CUtensorMap *map, const void *base, const uint64_t dims[3], const uint64_t strides_bytes[2],
                             const uint32_t box[3]);

// Floats of segment workspace that GEMMs of up to max_tiles tiles on up to max_n_pad nodes need.
size_t gemm_tc_partial_floats(int n_sms, int max_tiles, int max_n_pad);

// Describes one GEMM (fills everything but items_per_cta and grid, which the launcher sets).
GemmDesc make_gemm_desc(int n_in, const EpiParams &ep, const void *w_tiled = nullptr, bool w4 = false);

// Fixes how the GEMM is cut up (k-blocks per ring item, items per CTA, grid); launch_gemm_tc calls it itself.
cudaError_t plan_gemm_tc(GemmParams &p, int n_sms);

// Enqueues one GEMM: the streaming kernel, then the finishing kernel (both with programmatic
// stream serialization). partial_floats is the size of p.partials; cudaErrorInvalidValue if the
// GEMM needs more. *launched (optional) receives the number of kernels enqueued.
cudaError_t launch_gemm_tc(const GemmMaps &maps, GemmParams &p, int n_sms, size_t partial_floats, cudaStream_t st, int *launched);

}  // namespace llmcad
