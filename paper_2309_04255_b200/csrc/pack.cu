// One-time re-layout of a weight matrix for the tensor-core GEMM: row-major bf16 [n_out][n_in]
// becomes a sequence of 16 KB tiles (128 rows x 64 columns), tile-row major then k-block, each
// tile stored exactly as the MMA wants it in shared memory (128-byte rows, the 16-byte chunk c of
// row r at chunk position c ^ (r & 7): the 128-byte swizzle). A tile is then one contiguous 16 KB
// run in HBM that a single bulk copy moves into the ring: the copy engine issues a few large
// requests instead of 128 row-sized ones, and DRAM sees whole pages. Rows and columns past the
// matrix are zero.
#include "common.cuh"

namespace llmcad {

__global__ void tile_weight_kernel(const uint4 *__restrict__ src, int n_out, int n_in, int kb_per_tile, long long n_chunks,
                                   uint4 *__restrict__ dst)
{
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;   // one 16-byte chunk of the output
    if (idx >= n_chunks) return;
    const int pos = (int)(idx & 7);           // chunk position inside the 128-byte row
    const int r = (int)((idx >> 3) & 127);    // row inside the tile
    const long long tk = idx >> 10;           // tile * kb_per_tile + kb
    const int kb = (int)(tk % kb_per_tile);
    const int tile = (int)(tk / kb_per_tile);
    const int c = pos ^ (r & 7);              // logical chunk stored at this position
    const int row = tile * 128 + r, col = kb * 64 + c * 8;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (row < n_out && col < n_in) v = src[((size_t)row * n_in + col) >> 3];   // n_in is a multiple of 8
    dst[idx] = v;
}

size_t tiled_weight_bytes(int n_out, int n_in)
{
    return (size_t)((n_out + 127) / 128) * ((n_in + 63) / 64) * 16384;
}

cudaError_t launch_tile_weight(const void *w, int n_out, int n_in, void *dst, cudaStream_t st)
{
    const int kbpt = (n_in + 63) / 64;
    const long long n_chunks = (long long)((n_out + 127) / 128) * kbpt * 1024;
    const int block = 256;
    tile_weight_kernel<<<(unsigned)((n_chunks + block - 1) / block), block, 0, st>>>((const uint4 *)w, n_out, n_in, kbpt, n_chunks,
                                                                                   (uint4 *)dst);
    return cudaGetLastError();
}

}  // namespace llmcad
