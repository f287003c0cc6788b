// Micro-benchmarks behind the design notes (measurement interface, include/llmcad_profile.h): what the
// machine gives to the two access patterns the verification pass is made of.
//
// llmcad_probe_bulk_copy: one thread per CTA, one CTA per SM, streams its share of a buffer from HBM into
// shared memory with cp.async.bulk copies of a given size, a given number of them in flight: the ceiling
// of the weight stream of the skinny GEMMs (gemm_tc.cu), without any consumer.
// llmcad_probe_mma_sync: rate and latency of the legacy mma.sync.m16n8k16 bf16 path that the attention
// kernel for small trees runs on (attention_tc.cu).
#include <cuda_runtime.h>

#include <cstdint>
#include <vector>

#include "../../include/llmcad_profile.h"
#include "common.cuh"

namespace llmcad {
namespace {

constexpr int kMaxInFlight = 16;

__device__ __forceinline__ uint32_t probe_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// out[2 * cta] = ns from the first copy issued to the last copy landed, out[2 * cta + 1] = summed latency of the copies
__global__ void bulk_copy_probe_kernel(const uint8_t *src, size_t per_cta, int copy_bytes, int in_flight, int copies,
                                       unsigned long long *out, unsigned long long wait_limit_ns, int32_t *status)
{
    extern __shared__ __align__(1024) uint8_t probe_sm[];
    __shared__ uint64_t bar[kMaxInFlight];
    if (threadIdx.x != 0) return;
    for (int i = 0; i < in_flight; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(probe_smem_u32(&bar[i])));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    const uint8_t *base = src + (size_t)blockIdx.x * per_cta;
    const uint64_t t0 = global_timer_ns();
    unsigned long long lat_sum = 0;
    uint64_t issued_at[kMaxInFlight];
    bool gave_up = false;
    for (int i = 0; i < copies + in_flight && !gave_up; ++i) {
        const int s = i % in_flight;
        if (i >= in_flight) {
            const uint32_t par = ((uint32_t)(i / in_flight) - 1u) & 1u;
            uint32_t ok = 0;
            for (uint32_t spin = 0; !ok; ++spin) {
                asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                             : "=r"(ok) : "r"(probe_smem_u32(&bar[s])), "r"(par) : "memory");
                if (!ok && (spin & 1023u) == 1023u && global_timer_ns() - issued_at[s] > wait_limit_ns) { gave_up = true; break; }
            }
            if (gave_up) break;
            lat_sum += global_timer_ns() - issued_at[s];
        }
        if (i < copies) {
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(probe_smem_u32(&bar[s])), "r"(copy_bytes) : "memory");
            issued_at[s] = global_timer_ns();
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                         ::"r"(probe_smem_u32(probe_sm) + (uint32_t)s * (uint32_t)copy_bytes), "l"(base + (size_t)i * copy_bytes), "r"(copy_bytes),
                           "r"(probe_smem_u32(&bar[s])), "l"(pol) : "memory");
        }
    }
    if (gave_up) {
        atomicCAS(status, 0, LLMCAD_ERR_TIMEOUT);
        // let what is still on its way land before the shared memory goes away
        const uint64_t t1 = global_timer_ns();
        while (global_timer_ns() - t1 < 2000000ull) __nanosleep(1000);
    }
    out[2 * blockIdx.x] = global_timer_ns() - t0;
    out[2 * blockIdx.x + 1] = lat_sum;
}

__device__ __forceinline__ void probe_mma(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

template <int ACC>
__global__ void mma_sync_probe_kernel(float *sink, long long *cycles, int iters)
{
    float d[ACC][4];
#pragma unroll
    for (int i = 0; i < ACC; ++i) d[i][0] = d[i][1] = d[i][2] = d[i][3] = 0.f;
    const uint32_t a[4] = {threadIdx.x, 2u, 3u, 4u};
    const uint32_t b0 = threadIdx.x * 7u, b1 = 9u;
    __syncthreads();
    const long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < ACC; ++i) probe_mma(d[i], a, b0, b1);
    }
    const long long t1 = clock64();
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < ACC; ++i) s += d[i][0] + d[i][1] + d[i][2] + d[i][3];
    sink[blockIdx.x * blockDim.x + threadIdx.x] = s;
    if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

}  // namespace
}  // namespace llmcad

using namespace llmcad;

extern "C" int llmcad_probe_bulk_copy(const void *src, size_t bytes, int32_t copy_bytes, int32_t in_flight, void *stream,
                                      double *gbs, double *latency_us)
{
    if (src == nullptr || gbs == nullptr || latency_us == nullptr) return LLMCAD_ERR_INVALID_ARG;
    if (copy_bytes < 16 || copy_bytes % 16 || in_flight < 1 || in_flight > kMaxInFlight) return LLMCAD_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(src) & 15) != 0) return LLMCAD_ERR_INVALID_ARG;
    const size_t ring = (size_t)copy_bytes * in_flight;
    if (ring > 200 * 1024) return LLMCAD_ERR_INVALID_ARG;
    int dev = 0, n_sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return LLMCAD_ERR_CUDA;
    const long long copies = (long long)(bytes / ((size_t)n_sms * copy_bytes));
    if (copies < in_flight || copies > (1 << 30)) return LLMCAD_ERR_INVALID_ARG;
    const size_t per_cta = (size_t)copies * copy_bytes;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned long long *out = nullptr;
    int32_t *status = nullptr;
    if (cudaMalloc(&out, (size_t)n_sms * 2 * sizeof(unsigned long long) + sizeof(int32_t) * 4) != cudaSuccess) return LLMCAD_ERR_CUDA;
    status = reinterpret_cast<int32_t *>(out + (size_t)n_sms * 2);
    int rc = LLMCAD_OK;
    std::vector<unsigned long long> h((size_t)n_sms * 2);
    int32_t hs = 0;
    if (cudaMemsetAsync(status, 0, sizeof(int32_t), st) != cudaSuccess ||
        cudaFuncSetAttribute(bulk_copy_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(ring + 1024)) != cudaSuccess) rc = LLMCAD_ERR_CUDA;
    if (rc == LLMCAD_OK) {
        bulk_copy_probe_kernel<<<n_sms, 32, ring + 1024, st>>>(static_cast<const uint8_t *>(src), per_cta, copy_bytes, in_flight, (int)copies, out,
                                                               kDefaultWaitLimitNs, status);
        if (cudaGetLastError() != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess ||
            cudaMemcpy(h.data(), out, h.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost) != cudaSuccess ||
            cudaMemcpy(&hs, status, sizeof hs, cudaMemcpyDeviceToHost) != cudaSuccess) rc = LLMCAD_ERR_CUDA;
    }
    cudaFree(out);
    if (rc != LLMCAD_OK) return rc;
    if (hs != 0) return hs;
    double t_max = 0.0, lat = 0.0;
    for (int i = 0; i < n_sms; ++i) {
        if ((double)h[2 * i] > t_max) t_max = (double)h[2 * i];
        lat += (double)h[2 * i + 1] / (double)copies;
    }
    *gbs = (double)n_sms * (double)per_cta / t_max;          // bytes per ns = GB/s
    *latency_us = lat / n_sms / 1e3;
    return LLMCAD_OK;
}

extern "C" int llmcad_probe_mma_sync(int32_t warps, int32_t accumulators, void *stream, double *fma_per_clk_sm, double *cycles_per_mma)
{
    if (fma_per_clk_sm == nullptr || cycles_per_mma == nullptr || warps < 1 || warps > 32) return LLMCAD_ERR_INVALID_ARG;
    if (accumulators != 1 && accumulators != 2 && accumulators != 4 && accumulators != 8) return LLMCAD_ERR_INVALID_ARG;
    int dev = 0, n_sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return LLMCAD_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int threads = warps * 32, iters = 2000;
    float *sink = nullptr;
    if (cudaMalloc(&sink, (size_t)n_sms * threads * sizeof(float) + (size_t)n_sms * sizeof(long long)) != cudaSuccess) return LLMCAD_ERR_CUDA;
    long long *cyc = reinterpret_cast<long long *>(sink + (size_t)n_sms * threads);
    int rc = LLMCAD_OK;
    for (int rep = 0; rep < 2 && rc == LLMCAD_OK; ++rep) {        // the second run counts
        switch (accumulators) {
        case 1: mma_sync_probe_kernel<1><<<n_sms, threads, 0, st>>>(sink, cyc, iters); break;
        case 2: mma_sync_probe_kernel<2><<<n_sms, threads, 0, st>>>(sink, cyc, iters); break;
        case 4: mma_sync_probe_kernel<4><<<n_sms, threads, 0, st>>>(sink, cyc, iters); break;
        default: mma_sync_probe_kernel<8><<<n_sms, threads, 0, st>>>(sink, cyc, iters); break;
        }
        if (cudaGetLastError() != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess) rc = LLMCAD_ERR_CUDA;
    }
    long long h = 0;
    if (rc == LLMCAD_OK && cudaMemcpy(&h, cyc, sizeof h, cudaMemcpyDeviceToHost) != cudaSuccess) rc = LLMCAD_ERR_CUDA;
    cudaFree(sink);
    if (rc != LLMCAD_OK) return rc;
    if (h <= 0) return LLMCAD_ERR_CUDA;
    *cycles_per_mma = (double)h / ((double)iters * accumulators);
    *fma_per_clk_sm = (double)warps * iters * accumulators * 2048.0 / (double)h;      // m16n8k16: 2048 multiply-adds
    return LLMCAD_OK;
}
