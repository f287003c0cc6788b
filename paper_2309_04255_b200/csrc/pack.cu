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

// ------------------------------------------------------------------------------------------------
// INT4 weights (Sec. 4.1: the target model's weights are held as INT4 through group-wise
// quantisation). Format of this library: symmetric codes q in [-8, 7], one power-of-two scale 2^e per
// row and group of 64 input columns (= one k-block), e the smallest integer with max|w| <= 7 * 2^e,
// q = w / 2^e rounded to nearest, halves to even. q * 2^e is exact in bf16, so the GEMM computes with
// the dequantised weights exactly.
//
// One group: x[0..63] bf16 -> codes (offset binary u = q + 8) and the exponent.
__device__ __forceinline__ int quantize_group64(const uint4 (&raw)[8], uint32_t (&u)[64])
{
    float w[64];
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        const uint32_t v[4] = {raw[c].x, raw[c].y, raw[c].z, raw[c].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            w[c * 8 + 2 * j] = __uint_as_float(v[j] << 16);
            w[c * 8 + 2 * j + 1] = __uint_as_float(v[j] & 0xffff0000u);
        }
    }
    float m = 0.f;
#pragma unroll
    for (int i = 0; i < 64; ++i) m = fmaxf(m, fabsf(w[i]));
    int e = -126;
    if (m > 0.f) {
        int k;
        const float f = frexpf(m, &k);            // m = f * 2^k, f in [0.5, 1); 7 * 2^e = 0.875 * 2^(e + 3)
        e = (f <= 0.875f) ? k - 3 : k - 2;
        if (e < -126) e = -126;
    }
#pragma unroll
    for (int i = 0; i < 64; ++i) {
        float v = rintf(scalbnf(w[i], -e));       // exact scaling, then to nearest with halves to even
        v = fminf(fmaxf(v, -8.f), 7.f);
        u[i] = (uint32_t)((int)v + 8);
    }
    return e;
}

// Plain arrays, for inspection: q [n_out][n_in] int8 in [-8, 7], e [n_out][n_in / 64] int8.
__global__ void quantize_int4_plain_kernel(const uint4 *__restrict__ w, int n_out, int n_in, int8_t *__restrict__ q,
                                           int8_t *__restrict__ e)
{
    const int groups = n_in / 64;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;   // one (row, group)
    if (idx >= (long long)n_out * groups) return;
    const int row = (int)(idx / groups), g = (int)(idx % groups);
    uint4 raw[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) raw[c] = w[((size_t)row * n_in + (size_t)g * 64) / 8 + c];
    uint32_t u[64];
    const int ex = quantize_group64(raw, u);
    e[idx] = (int8_t)ex;
#pragma unroll
    for (int i = 0; i < 64; ++i) q[(size_t)row * n_in + (size_t)g * 64 + i] = (int8_t)((int)u[i] - 8);
}

// The layout the GEMM streams: per (tile of 128 rows, k-block of 64 columns) 4224 bytes: 128 rows x 8
// words of eight codes each (word c of row r = columns 8c .. 8c+7, element j of the word in the nibble
// at bit 4 * (j / 2) + 16 * (j % 2), so that (word >> 4k) & 0x000f000f holds elements 2k and 2k + 1 in
// its two halves), then the 128 exponents of the rows. Tiles in the order [tile][k-block]. Rows past
// the matrix are zero (code 8 = 0, exponent -126).
__global__ void tile_weight_int4_kernel(const uint4 *__restrict__ w, int n_out, int n_in, int kb_per_tile, long long n_rows,
                                        uint8_t *__restrict__ dst)
{
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;   // one row of one (tile, k-block)
    if (idx >= n_rows) return;
    const int r = (int)(idx & 127);
    const long long tk = idx >> 7;
    const int kb = (int)(tk % kb_per_tile), tile = (int)(tk / kb_per_tile);
    const int row = tile * 128 + r;
    uint8_t *t = dst + (size_t)tk * kW4TileBytes;
    uint32_t words[8];
    int ex = -126;
    if (row < n_out) {
        uint4 raw[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) raw[c] = w[((size_t)row * n_in + (size_t)kb * 64) / 8 + c];
        uint32_t u[64];
        ex = quantize_group64(raw, u);
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            uint32_t x = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) x |= u[c * 8 + j] << (4 * (j >> 1) + 16 * (j & 1));
            words[c] = x;
        }
    } else {
#pragma unroll
        for (int c = 0; c < 8; ++c) words[c] = 0x88888888u;
    }
    uint4 *tw = reinterpret_cast<uint4 *>(t) + (size_t)r * 2;
    tw[0] = make_uint4(words[0], words[1], words[2], words[3]);
    tw[1] = make_uint4(words[4], words[5], words[6], words[7]);
    reinterpret_cast<int8_t *>(t + 4096)[r] = (int8_t)ex;
}

size_t tiled_weight_int4_bytes(int n_out, int n_in)
{
    return (size_t)((n_out + 127) / 128) * (n_in / 64) * kW4TileBytes;
}

cudaError_t launch_quantize_int4_plain(const void *w, int n_out, int n_in, int8_t *q, int8_t *e, cudaStream_t st)
{
    const long long n = (long long)n_out * (n_in / 64);
    quantize_int4_plain_kernel<<<(unsigned)((n + 127) / 128), 128, 0, st>>>((const uint4 *)w, n_out, n_in, q, e);
    return cudaGetLastError();
}

cudaError_t launch_tile_weight_int4(const void *w, int n_out, int n_in, void *dst, cudaStream_t st)
{
    const int kbpt = n_in / 64;
    const long long n_rows = (long long)((n_out + 127) / 128) * kbpt * 128;
    tile_weight_int4_kernel<<<(unsigned)((n_rows + 127) / 128), 128, 0, st>>>((const uint4 *)w, n_out, n_in, kbpt, n_rows, (uint8_t *)dst);
    return cudaGetLastError();
}

}  // namespace llmcad
